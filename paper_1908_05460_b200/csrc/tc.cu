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
// A CTA owns one (k-tile, c-tile) block of dW and a contiguous range of reduction chunks.  Consecutive
// splits form a thread-block cluster and add their blocks through distributed shared memory; if a tile
// has several clusters, each cluster leaves its sum in a slot of the workspace and a second, small kernel
// (reduce_slots_kernel, launched as a programmatic dependent so its start-up overlaps) adds the slots with
// the whole GPU, in an order that depends only on the launch geometry.  No CTA waits for a CTA outside
// its cluster.  (Summing in the same kernel -- by the last cluster to arrive, or by all CTAs of a tile
// once a counter shows them complete -- measured slower: the first serialises megabytes of slot reads on
// a few CTAs, the second needs the whole grid resident, which cluster placement does not guarantee.)
//
// Warp roles: warp 0 = TMA producer (the whole warp: lane b issues copy b of a stage, so the per-copy issue
// cost overlaps); warps 1..3 = MMA issuers (one elected thread each; warp 1 also owns the TMEM allocation);
// all eight warps run the epilogue.  The filter rows are dealt round-robin to the issuers: a single thread
// sustains only one small MMA per ~100 cycles, and rows accumulate independently.  A CTA that holds a single
// filter row keeps TWO accumulators for it: two issuers take alternate chunks of the reduction, and the
// epilogue adds accumulator 0 + accumulator 1 (a fixed order).
//
// Small maps (at most 16 pixels): both operands are MN-major with 128-byte rows of 64 channels (dY through a
// transposed copy), the reduction index is ordered (pixel, image) through tensor maps with permuted dimensions,
// and a chunk's X arrives as one haloed tile, so a filter shift is again a descriptor offset.
//
// fp32 inputs: kind::tf32 on operands split into two planes (the upper mantissa bits and the remainder), three
// MMAs per k-step (big*big + big*small + small*big); an MN-major 32-bit operand uses the 128-byte swizzle on
// 32-byte units.  One plain TF32 pass on request.
//
// Every mbarrier wait is bounded; on expiry the kernel raises the workspace status word, drains
// the copies it has in flight, frees its tensor memory and returns.
#include <cuda.h>

#include <cooperative_groups.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "gaconv_internal.h"
#include "tma.cuh"

// GACONV_TUNING builds carry clock64 stamps of CTA (0,0)'s phases (workspace bytes [64,128)) and read
// planner overrides from the environment; the default build has neither.
#ifdef GACONV_TUNING
#define GACONV_TL(slot, cond) do { if (tl && (cond)) tl[slot] = clock64(); if (P.timeline && threadIdx.x == 128) gaconv_tuning_stamps[(blockIdx.y * gridDim.x + blockIdx.x) & 1023][slot] = gaconv_globaltimer(); } while (0)
__device__ unsigned long long gaconv_tuning_stamps[1024][8];
// per launch (CTA (0,0)): {entry, dependency satisfied, exit, shape} in nanoseconds of the global timer
__device__ unsigned long long gaconv_tuning_tc_log[4096][4];
__device__ unsigned int gaconv_tuning_tc_log_n;
__device__ __forceinline__ unsigned long long gaconv_globaltimer() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
#else
#define GACONV_TL(slot, cond) do { } while (0)
#endif

namespace gaconv {
namespace {

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_bf16_acc(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, 1, 1;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc) : "memory");
}
// 16 bytes from the same shared-memory offset in CTA `rank` of this cluster
__device__ __forceinline__ float4 ld_dsmem_f4(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    float4 v;
    // not volatile: the blocks are stable between the two cluster barriers, so the compiler may batch these loads
    asm("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(remote));
    return v;
}
// fp32 operands read as TF32 (the tensor core takes the upper 19 bits of each word)
__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3, int c4) {
    asm volatile("cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Issues the load only; the caller executes tcgen05.wait::ld before reading v.
__device__ __forceinline__ void tmem_ld16_nowait(uint32_t taddr, float (&v)[16]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]),
                   "=f"(v[8]), "=f"(v[9]), "=f"(v[10]), "=f"(v[11]), "=f"(v[12]), "=f"(v[13]), "=f"(v[14]), "=f"(v[15])
                 : "r"(taddr));
}
struct TcParams {
    Geom g;
    int m;              // MMA M: 64 or 128 output channels per k-tile
    int kb;             // rows of an A box (k rounded up to 8, at most m)
    int ct;             // input channels per c-tile; MMA N = s * ct
    int ct_shift;       // log2(ct)
    int tiles_k, tiles_c, splits;
    int chunk_base, chunk_rem;   // split i takes chunk_base chunks, one more when i < chunk_rem
    int halo;           // 1: S tiles with R-1 halo rows, row shift = row offset; 0: R*S tiles
    int ci, bp;         // chunk = ci images x bp output rows (ci > 1: whole maps)
    int chunks;         // total chunks of the reduction
    int a_sub_px;       // pixels per A box = min(64, PQ)
    int a_subs;         // A boxes per chunk
    int a_subs_img;     // A boxes per image of a chunk (maps of 64 pixels and more)
    int a_sub_bytes;    // kb * a_sub_px * 2
    int a_region_bytes; // a_subs * a_sub_bytes rounded up to 1 KiB (B tiles start there)
    int a_swz, b_swz;   // swizzle codes of the descriptors
    int b_tiles;        // S (halo) or R*S; 1 when wide
    int tiny;           // 1: maps of fewer than 64 pixels: A comes from a transposed copy dYt[n][pq][k] (MN-major,
                        //    64 channels per 128-byte row); chunks are whole images, 16 reduction rows per k-step
    int tiny2;          // with tiny, for single-row CTAs of stride-1 layers: the reduction rows of a chunk of ci (8, 16 or 32) images
                        //    are ordered (pixel, image).  Then ONE X tile with a column halo, laid out [row][column][image][channel]
                        //    by a tensor map with permuted dimensions, serves all column shifts (a shift = one pixel = ci 128-byte
                        //    rows), as the wide tile does for maps of 64 pixels and more
    int b_lbo;          // B descriptor: bytes between the column-shift atoms of an MMA
    int b_sub_bytes;    // B descriptor advance from one A box (or image row) to the next
    int f32;            // 1: fp32 inputs on kind::tf32 MMAs (32-pixel A boxes, 32-channel B tiles, k-steps of 8 pixels).
                        //    passes == 3: the operands come as two planes each, big = the TF32 part of x and small = x - big,
                        //    and every k-step issues big*big + big*small + small*big into the same accumulator (fp32 accuracy);
                        //    passes == 1: the tensors themselves, cut to TF32 by the tensor core
    int passes;
    int kpx;            // pixels per k-step: 16 (bf16) or 8 (tf32)
    int a_plane_bytes, b_plane_bytes;   // distance from the big to the small plane inside a stage
    int by_image;       // 1: a chunk is ci whole images (maps under 64 pixels)
    int a_k4_step;      // descriptor advance (16-byte units) from one k-step to the next inside an A box
    int a_lbo;          // leading byte offset of the A descriptor
    int wide;           // 1: ONE tile of (rows + rc - 1) x (Q + S - 1) pixels; a column shift is a one-pixel
                        //    descriptor offset (leading byte offset = one pixel row), a row shift a whole tile row
    int b_tile_stride;  // bytes between consecutive B tiles (multiple of 1024)
    int b_tile_bytes;   // bytes one TMA writes per B tile
    int stage_bytes, stages;
    int ksteps;         // ci*bp*Q/16
    int tmem_cols;      // power of two >= 32
    int cl;             // thread-block cluster size along the split dimension (1..4); divides splits
    int rsplit;         // 1: a CTA handles ONE filter row (tile index carries r); N = s * 64
    int rc;             // filter rows per CTA: g.r, or 1 when rsplit
    int dual;           // 1 (only with rc == 1): two accumulators, issuer i takes the chunks with (index & 1) == i
    int stack;          // 1: the R filter rows are stacked in M (row r of the filter = rows r*kb .. r*kb+kb-1 of the accumulator):
                        //    A = R copies of the dY box, shifted by one image row each; B = the X rows of the chunk, no halo rows
    int issuers;        // MMA-issuing warps: min(R, 3), or 2 when dual; issuer i takes filter rows i, i+issuers, ...
    int slot_quads;     // float4 elements of one cluster slot (m rows x rc * s * ct columns)
    uint32_t qpr_magic; // ceil(2^32 / quads per row): quad index -> row by one multiply
    int reduce_parts;   // grid.x of reduce_slots_kernel
    uint32_t idesc;
    int timeline;       // tuning builds: CTA (0,0) records clock64 stamps of its phases at workspace bytes [64, 128)
};

constexpr int kMaxStages = 8;
// accumulator row -> element offset of its output channel (and, when the filter rows are stacked in M, its filter
// row) in dW; -1 for a row that holds nothing
__device__ __forceinline__ int tc_row_offset(const TcParams& P, int k0, int row)
{
    const Geom& g = P.g;
    if (!P.stack) return k0 + row < g.k ? (int)((k0 + row) * g.ws_k) : -1;
    const int r = row / P.kb, kk = row - r * P.kb;
    return (r < g.r && kk < g.k) ? (int)(kk * g.ws_k + r * g.ws_r) : -1;
}

constexpr int kMaxQuadCols = 7 * 256 / 4;      // rc <= 7 filter rows of at most 256 columns

// R_T: filter rows (0 = take it from the geometry); KS_T: k-steps per A box (0 = from the plan).
// The compile-time values let the issue loop unroll into straight-line MMA instructions.
template <int R_T, int KS_T>
__global__ void __launch_bounds__(256, 1)
exact_tc_kernel(const __grid_constant__ CUtensorMap map_dy, const __grid_constant__ CUtensorMap map_x,
                float* __restrict__ dw, float* __restrict__ partial, uint32_t* __restrict__ counters,
                uint32_t* __restrict__ status, const TcParams P)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[kMaxStages], bar_empty[kMaxStages], bar_acc;
    __shared__ uint32_t s_tmem_base;
    __shared__ volatile int s_abort;
    // for quad column cq of the CTA's block: offset of its first element within a dW row block, and how many of
    // its four channels exist (the last channel tile may be partial)
    __shared__ int s_coloff[kMaxQuadCols];
    __shared__ signed char s_colvalid[kMaxQuadCols];
    __shared__ int s_rowoff[128];              // accumulator row -> offset in dW, or -1

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Geom& g = P.g;

    const int tile = blockIdx.x, split = blockIdx.y;
    const int r_lo = P.rsplit ? tile % g.r : 0;                 // first filter row of this CTA
    const int kc_tile = P.rsplit ? tile / g.r : tile;
    const int k0 = (kc_tile / P.tiles_c) * P.m, c0 = (kc_tile % P.tiles_c) * P.ct;
    const int ch_begin = split * P.chunk_base + min(split, P.chunk_rem);
    const int nchunks = P.chunk_base + (split < P.chunk_rem ? 1 : 0);
    const int nmma = g.s * P.ct;
    float* red = reinterpret_cast<float*>(smem_raw + (smem_base - smem_u32(smem_raw)));   // reduction block, aliases the stages
    const int red_stride = P.rc * nmma + 4;

#ifdef GACONV_TUNING
    if (P.timeline && threadIdx.x == 128) gaconv_tuning_stamps[(blockIdx.y * gridDim.x + blockIdx.x) & 1023][1] = gaconv_globaltimer();
#endif
    pdl_release_next_grid();
    if (threadIdx.x < P.m) s_rowoff[threadIdx.x] = tc_row_offset(P, k0, threadIdx.x);
    const int acc_rows = P.stack ? g.r * P.kb : min(P.m, g.k - k0);          // accumulator rows in use
    for (int cq = threadIdx.x; cq < (P.rc * nmma) >> 2; cq += blockDim.x) {
        const int col = cq << 2, rl = col / nmma, sc = col - rl * nmma, s_ = sc >> P.ct_shift, c = c0 + (sc & (P.ct - 1));
        s_coloff[cq] = (int)((r_lo + rl) * g.ws_r + s_ * g.ws_s + c * g.ws_c);
        s_colvalid[cq] = (signed char)max(0, min(4, g.c - c));
    }
    if (threadIdx.x == 0) {
        // the tensor maps are kernel parameters: fetching them does not depend on the previous kernel
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_dy) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        for (int i = 0; i < P.stages; ++i) { mbar_init(smem_u32(&bar_full[i]), 1); mbar_init(smem_u32(&bar_empty[i]), P.dual ? 1 : P.issuers); }
        mbar_init(smem_u32(&bar_acc), P.issuers);
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
#ifdef GACONV_TUNING
    const unsigned long long t_in = gaconv_globaltimer();
#endif
    pdl_wait_prior_grid();     // set-up done; from here on global memory of the previous kernel is read and written
#ifdef GACONV_TUNING
    __shared__ unsigned int s_log_i;
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
        s_log_i = atomicAdd(&gaconv_tuning_tc_log_n, 1u) & 4095u;
        gaconv_tuning_tc_log[s_log_i][0] = t_in; gaconv_tuning_tc_log[s_log_i][1] = gaconv_globaltimer();
        gaconv_tuning_tc_log[s_log_i][3] = ((unsigned long long)g.c << 40) | ((unsigned long long)g.k << 24) | ((unsigned long long)gridDim.x * gridDim.y << 8) | (unsigned)g.p;
    }
#endif
#ifdef GACONV_TUNING
    long long* tl = (P.timeline && blockIdx.x == 0 && blockIdx.y == 0) ? reinterpret_cast<long long*>(status + 16) : nullptr;
#endif
    GACONV_TL(0, threadIdx.x == 0);

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (whole warp)
        // Lane 0 waits for the stage and posts the byte count; then lane b issues copy b of the chunk, so the
        // copies of a stage leave together instead of one after the other from a single thread.
        // Chunk coordinates advance incrementally: no division inside the loop for the first 32 copies.
        int n0, p0;
        const bool whole_maps = P.by_image != 0 || P.ci > 1;
        const int cpi = whole_maps ? 1 : g.p / P.bp;
        if (whole_maps) { n0 = ch_begin * P.ci; p0 = 0; }
        else { n0 = ch_begin / cpi; p0 = (ch_begin % cpi) * P.bp; }
        const int planes = P.f32 && P.passes == 3 ? 2 : 1;
        const uint32_t tx_bytes = planes * ((P.tiny ? (P.m / 64) * P.ci * g.p * g.q * 128 : P.stack ? P.a_subs * g.r * P.kb * 128 : P.a_subs * P.a_sub_bytes) + P.b_tiles * P.b_tile_bytes);
        const int n_a = P.f32 ? planes * (P.stack ? g.r : 1) * P.a_subs : P.tiny ? P.m / 64 : P.by_image ? 1 : P.stack ? g.r * P.a_subs : P.a_subs, n_all = n_a + planes * P.b_tiles;
        // what copy `lane` is: image and box of an A copy, or filter row and column shift of a B copy
        const int a_img = (P.tiny || P.by_image) ? 0 : lane / P.a_subs_img, a_sub = (P.tiny || P.by_image) ? 0 : lane - a_img * P.a_subs_img;
        const int b_idx = lane - n_a, b_rr = b_idx > 0 ? b_idx / g.s : 0, b_ss = b_idx > 0 ? b_idx - b_rr * g.s : 0;
        int issued = 0, st = 0, ph = 0;
        for (int it = 0; it < nchunks; ++it) {
            const uint32_t full = smem_u32(&bar_full[st]);
            int ok = 1;
            if (lane == 0) {
                if (it >= P.stages && !mbar_wait(smem_u32(&bar_empty[st]), ph ^ 1)) { s_abort = 1; atomicOr(status, 1u); }
                if (s_abort) ok = 0;
                else mbar_expect_tx(full, tx_bytes);
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            const uint32_t sa = smem_base + st * P.stage_bytes;
            const uint32_t sb = sa + P.a_region_bytes;
            for (int b = lane; b < n_all; b += 32) {
                if (P.f32) {                                                     // fp32: boxes of 32 pixels, one set per plane
                    if (b < n_a) {
                        const int per_plane = (P.stack ? g.r : 1) * P.a_subs;   // (stacked: one box per filter row, one image row earlier each)
                        const int pl = b / per_plane, rest = b - pl * per_plane, rr = rest / P.a_subs, sub = rest - rr * P.a_subs;
                        const int i = sub / P.a_subs_img, sb_ = sub - i * P.a_subs_img;
                        tma_load_4d(sa + pl * P.a_plane_bytes + sub * P.a_sub_bytes + rr * P.kb * 128, &map_dy, full,
                                    (P.stack ? p0 - rr + g.pad_h : p0) * g.q + P.a_sub_px * sb_, k0, n0 + i, pl);
                    } else {
                        const int pl = b - n_a;
                        tma_load_5d(sb + pl * P.b_plane_bytes, &map_x, full, c0, -g.pad_w, P.stack ? p0 : p0 + r_lo - g.pad_h, n0, pl);
                    }
                } else if (b < n_a) {
                    if (P.tiny2) {                                               // one box per 64-channel atom, [pixel][image][k]
                        tma_load_3d(sa + b * P.a_lbo, &map_dy, full, k0 + 64 * b, n0, 0);
                    } else if (P.tiny) {                                         // one box per 64-channel atom, [image][pixel][k]
                        tma_load_3d(sa + b * P.a_lbo, &map_dy, full, k0 + 64 * b, 0, n0);
                    } else if (P.by_image) {
                        tma_load_3d(sa, &map_dy, full, 0, k0, n0);               // ci whole maps in one box
                    } else if (P.stack) {                                        // filter row rr: the box one image row earlier per row;
                        const int rr = b / P.a_subs, sb_ = b - rr * P.a_subs;    // rows that leave the map read as zeros
                        const int i = sb_ / P.a_subs_img, sub = sb_ - i * P.a_subs_img;
                        tma_load_3d(sa + sb_ * P.a_sub_bytes + rr * P.kb * 128, &map_dy, full, (p0 - rr + g.pad_h) * g.q + 64 * sub, k0, n0 + i);
                    } else {                                                     // images past the batch read as zeros
                        const int i = b < 32 ? a_img : b / P.a_subs_img, sub = b < 32 ? a_sub : b - i * P.a_subs_img;
                        tma_load_3d(sa + b * P.a_sub_bytes, &map_dy, full, p0 * g.q + 64 * sub, k0, n0 + i);
                    }
                } else {
                    const int j = b - n_a;
                    if (P.tiny2) {                                               // dimensions (c, n, w, h)
                        tma_load_4d(sb, &map_x, full, c0, n0, -g.pad_w, r_lo - g.pad_h);
                    } else if (P.wide) {
                        tma_load_4d(sb, &map_x, full, c0, -g.pad_w, P.stack ? p0 : p0 + r_lo - g.pad_h, n0);
                    } else if (P.halo) {
                        tma_load_4d(sb + j * P.b_tile_stride, &map_x, full, c0, j - g.pad_w, p0 - g.pad_h, n0);
                    } else {
                        const int rr = b < 32 ? b_rr : j / g.s, ss = b < 32 ? b_ss : j - rr * g.s;
                        tma_load_4d(sb + j * P.b_tile_stride, &map_x, full, c0, ss - g.pad_w, p0 * g.stride_h + r_lo + rr - g.pad_h, n0);
                    }
                }
            }
            ++issued;
            if (whole_maps) n0 += P.ci;
            else { p0 += P.bp; if (p0 >= g.p) { p0 = 0; ++n0; } }
            if (++st == P.stages) { st = 0; ph ^= 1; }
        }
        if (lane == 0 && s_abort) {   // drain: wait (bounded) for the copies already issued
            for (int it = max(0, issued - P.stages); it < issued; ++it) mbar_wait(smem_u32(&bar_full[it % P.stages]), (it / P.stages) & 1);
        }
    } else if (warp >= 1 && warp <= 3 && warp - 1 < P.issuers && lane == 0) {
        const int issuer = warp - 1;
        // ------------------------------------------------------------------ MMA issuer
        // descriptors are assembled from a constant high word and a low word that only advances
        const uint32_t eb = P.f32 ? 4u : 2u;
        const uint32_t a_row_bytes = P.tiny ? 128u : P.a_sub_px * eb, b_row_bytes = P.ct * eb;
        const uint32_t a_hi = ((8 * a_row_bytes) >> 4) | (1u << 14) | ((uint32_t)P.a_swz << 29);
        const uint32_t wt = g.q + g.s - 1;                       // pixels per tile row in wide mode
        // stride between the two 8-pixel halves of a k-step: contiguous, except in wide mode when a k-step spans two rows
        // (fp32: an MN-major tf32 operand uses the 128-byte swizzle on 32-byte units, whose K groups are 4 pixels)
        const uint32_t b_sbo = P.f32 ? 4 * b_row_bytes : (P.wide && g.q == 8) ? wt * b_row_bytes : 8 * b_row_bytes;
        const uint32_t b_hi = (b_sbo >> 4) | (1u << 14) | ((uint32_t)P.b_swz << 29);
        const uint32_t a_lo_c = (((uint32_t)P.a_lbo >> 4) & 0x3fffu) << 16, b_lo_c = (((uint32_t)P.b_lbo >> 4) & 0x3fffu) << 16;
        const int ks_per_sub = P.a_sub_px / P.kpx;
        const uint32_t a_k4 = (uint32_t)P.a_k4_step;
        const uint32_t a_sub_step = (uint32_t)P.a_sub_bytes >> 4;
        const uint32_t b_r_step = (P.wide ? wt * b_row_bytes : P.halo ? (uint32_t)g.q * b_row_bytes : (uint32_t)g.s * P.b_tile_stride) >> 4;
        // descriptor offset of k-step k4 inside an A box, and the advance from one A box to the next
        uint32_t b_k_off[4];
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4)
            b_k_off[k4] = (P.wide ? ((((uint32_t)P.kpx * k4) / g.q) * wt + ((uint32_t)P.kpx * k4) % g.q) * b_row_bytes : (uint32_t)P.kpx * k4 * b_row_bytes) >> 4;
        const uint32_t b_sub_step = (uint32_t)P.b_sub_bytes >> 4;
        const int R = R_T ? R_T : P.rc;
        const int KS = KS_T ? KS_T : ks_per_sub;
        // this issuer's filter rows: TMEM address of the accumulator and descriptor offset of the row
        constexpr int RI = R_T == 0 ? 3 : (R_T + 2) / 3;           // rows per issuer, at most (R <= 7 -> 3)
        uint32_t d_row[RI], b_row[RI];
        int nrows = 0;
#pragma unroll
        for (int i = 0; i < RI; ++i) {
            const int r = issuer + i * P.issuers;                   // dual: accumulator index, both on filter row 0 of the CTA
            d_row[i] = P.m == 128 ? tmem_base + r * nmma : tmem_base + (((uint32_t)(r & 1) * 16u) << 16) + (r >> 1) * nmma;
            b_row[i] = P.dual ? 0u : r * b_r_step;
            if (P.dual ? i == 0 : r < R) nrows = i + 1;
        }
        const uint64_t a_hi64 = (uint64_t)a_hi << 32, b_hi64 = (uint64_t)b_hi << 32;
        const uint32_t idesc = P.idesc;
        const int mine = P.dual ? issuer : 0, it_step_mask = P.dual ? 1 : 0;
        const uint32_t a_small = (uint32_t)P.a_plane_bytes >> 4, b_small = (uint32_t)P.b_plane_bytes >> 4;      // fp32, three passes
        int st = 0, ph = 0;
        bool fresh = true;            // the next k-step starts the accumulation (overwrites TMEM)
        for (int it = 0; it < nchunks; ++it) {
            if ((it & it_step_mask) == mine) {
                if (!mbar_wait(smem_u32(&bar_full[st]), ph)) { s_abort = 1; atomicOr(status, 1u); break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                GACONV_TL(1, it == 0 && issuer == 0);
                const uint32_t sa = smem_base + st * P.stage_bytes;
                // 14-bit start-address fields: in a cluster launch shared addresses carry the CTA rank in high bits
                uint32_t a_lo = a_lo_c | ((sa >> 4) & 0x3fffu);
                uint32_t b_lo = b_lo_c | (((sa + P.a_region_bytes) >> 4) & 0x3fffu);
                if (P.f32) {
                    // fp32 inputs: one accumulator per issuer (dual), k-steps of eight pixels; with split operands
                    // big*big, then the two cross terms, every k-step
                    for (int sub = 0; sub < P.a_subs; ++sub, a_lo += a_sub_step, b_lo += b_sub_step) {
#pragma unroll
                        for (int k4 = 0; k4 < 4; ++k4) {
                            if (k4 >= KS) break;
                            const uint64_t ad = a_hi64 | (a_lo + a_k4 * k4), bd = b_hi64 | (b_lo + b_k_off[k4]);
                            umma_tf32(d_row[0], ad, bd, idesc, fresh ? 0u : 1u);
                            fresh = false;
                            if (P.passes == 3) {
                                umma_tf32(d_row[0], ad, bd + b_small, idesc, 1u);
                                umma_tf32(d_row[0], ad + a_small, bd, idesc, 1u);
                            }
                        }
                    }
                } else
                for (int sub = 0; sub < P.a_subs; ++sub, a_lo += a_sub_step) {
                    if (fresh) {      // first k-step of this accumulator: accumulate flag off
#pragma unroll
                        for (int i = 0; i < RI; ++i)
                            if (i < nrows) umma_bf16(d_row[i], a_hi64 | a_lo, b_hi64 | (b_lo + b_row[i]), idesc, 0u);
                    }
#pragma unroll
                    for (int k4 = 0; k4 < KS; ++k4) {
                        if (!(fresh && k4 == 0)) {
#pragma unroll
                            for (int i = 0; i < RI; ++i)
                                if (i < nrows) umma_bf16_acc(d_row[i], a_hi64 | (a_lo + a_k4 * k4), b_hi64 | (b_lo + b_k_off[k4] + b_row[i]), idesc);
                        }
                    }
                    fresh = false;
                    b_lo += b_sub_step;
                }
                umma_commit(smem_u32(&bar_empty[st]));   // frees the stage once these MMAs have read it
            }
            if (++st == P.stages) { st = 0; ph ^= 1; }
        }
        umma_commit(smem_u32(&bar_acc));             // accumulators complete
        GACONV_TL(2, issuer == 0);
    }
    __syncwarp();
    const bool vec = g.ws_c == 1 && (g.c & 3) == 0;
    auto store_dw = [&](int row, int cq, const float4& t) {      // alpha * t -> the four elements of (row, quad column cq)
        const int ro = s_rowoff[row];
        if (ro < 0) return;
        float* p = dw + ro + s_coloff[cq];
        const int valid = s_colvalid[cq];
        const float a = g.alpha;
        if (vec && valid == 4) {
            *reinterpret_cast<float4*>(p) = make_float4(a * t.x, a * t.y, a * t.z, a * t.w);
        } else {
            const float tv[4] = {t.x, t.y, t.z, t.w};
            for (int j = 0; j < valid; ++j) p[(size_t)j * g.ws_c] = a * tv[j];
        }
    };
    {
        // ------------------------------------------------------------------ epilogue 1: TMEM -> shared memory
        // The accumulators go to a [row][column] fp32 block in this CTA's shared memory (the operand
        // stages are free by now); column = local filter row * nmma + s * ct + c.  Rows are padded by four
        // floats so that the 32 lanes of a warp, one row each, store 16-byte pieces without bank conflicts.
        // All eight warps take part (the producer and the issuers are done): warps w and w + 4 read the same
        // 32 lanes of tensor memory and take alternate 16-column pieces.
        const bool ready = mbar_wait_sleepy(smem_u32(&bar_acc), 0);
        if (!ready) { s_abort = 1; atomicOr(status, 1u); }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        GACONV_TL(3, threadIdx.x == 128);
        if (__all_sync(0xffffffffu, ready && !s_abort)) {       // warp-uniform: the tensor-memory loads are warp-wide
            const int sp = warp & 3, half = warp < 4 ? 1 : 0;
            const int row = P.m == 128 ? 32 * sp + lane : 16 * sp + (lane & 15);
            const uint32_t tlane = tmem_base + ((uint32_t)(32 * sp) << 16);
            const int pieces = nmma >> 4;                      // 16-column pieces per accumulator
            if (P.dual) {
                // accumulator 0 (even chunks) + accumulator 1 (odd chunks).  M = 128: they sit side by side in the
                // columns; M = 64: in the two 16-lane halves of each sub-partition (lane l and lane l + 16).
                const bool has0 = nchunks > 0, has1 = nchunks > 1;
                const bool row_ok = row < acc_rows && (P.m == 128 || lane < 16);
                float* rrow = red + row * red_stride;
                for (int pc = half; pc < pieces; pc += 4) {     // this warp: pieces pc and pc + 2
                    float v0[2][16], v1[2][16];
                    const int nld = pc + 2 < pieces ? 2 : 1;
#pragma unroll
                    for (int u = 0; u < 2; ++u)
                        if (u < nld) {
                            tmem_ld16_nowait(tlane + 16 * (pc + 2 * u), v0[u]);
                            if (P.m == 128) tmem_ld16_nowait(tlane + nmma + 16 * (pc + 2 * u), v1[u]);
                        }
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        if (u >= nld) continue;
                        float t[16];
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            const float a0 = v0[u][e];
                            const float a1 = P.m == 128 ? v1[u][e] : __shfl_down_sync(0xffffffffu, a0, 16);
                            t[e] = (has0 ? a0 : 0.f) + (has1 ? a1 : 0.f);
                        }
                        if (!row_ok) continue;
                        float4* p4 = reinterpret_cast<float4*>(rrow + 16 * (pc + 2 * u));
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) p4[q4] = make_float4(t[4 * q4], t[4 * q4 + 1], t[4 * q4 + 2], t[4 * q4 + 3]);
                    }
                }
            } else {
                const int groups = P.m == 128 ? P.rc : (P.rc + 1) / 2;
                for (int gi = 0; gi < groups; ++gi) {
                    const int rl = P.m == 128 ? gi : 2 * gi + (lane >> 4);      // row within this CTA's filter rows
                    const bool row_ok = rl < P.rc && k0 + row < g.k;
                    float* rrow = red + row * red_stride + rl * nmma;
                    for (int pc = half; pc < pieces; pc += 8) {                 // this warp: pieces pc, pc + 2, pc + 4, pc + 6
                        float v[4][16];                                        // up to four 16-column loads in flight
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            if (pc + 2 * u < pieces) tmem_ld16_nowait(tlane + gi * nmma + 16 * (pc + 2 * u), v[u]);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                        if (!row_ok) continue;
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            if (pc + 2 * u >= pieces) continue;
                            float4* p4 = reinterpret_cast<float4*>(rrow + 16 * (pc + 2 * u));
#pragma unroll
                            for (int q4 = 0; q4 < 4; ++q4) {
                                const float4 t4 = nchunks > 0 ? make_float4(v[u][4 * q4], v[u][4 * q4 + 1], v[u][4 * q4 + 2], v[u][4 * q4 + 3])
                                                              : make_float4(0.f, 0.f, 0.f, 0.f);
                                p4[q4] = t4;
                            }
                        }
                    }
                }
            }
        }
    }

    GACONV_TL(4, threadIdx.x == 128);
    // ---------------------------------------------------------------------- TMEM teardown
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(P.tmem_cols) : "memory");
    }

    // ---------------------------------------------------------------------- epilogue 2: split reduction
    // The cl CTAs of a cluster are consecutive splits of one output tile.  After a cluster barrier CTA
    // `rank` adds slice `rank` of the block over the cl CTAs through distributed shared memory, in
    // rank order.  With one cluster per tile the result (times alpha) goes straight to dW; with several,
    // to the cluster's slot in the workspace, which reduce_slots_kernel adds up afterwards.
    // A CTA that gave up on a wait still takes part in the barriers, so its peers never wait in vain.
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int cl = P.cl, rank = cl > 1 ? (int)cluster.block_rank() : 0;
    const int groups_per_tile = P.splits / cl, cgroup = split / cl;
    if (cl > 1) cluster.sync();
    GACONV_TL(5, threadIdx.x == 0);
    const int rows = acc_rows, cols = P.rc * nmma;
    const int q_per_row = cols >> 2, quads = rows * q_per_row;
    const int slice = (quads + cl - 1) / cl;
    const int f_begin = min(quads, rank * slice), f_end = min(quads, f_begin + slice);
    const bool direct = groups_per_tile == 1;
    // quad index -> (row, quad column) by a multiply with the rounded-up reciprocal (exact for these ranges), so the
    // iterations below are independent and the compiler keeps several quads in flight
    const uint32_t qpr_magic = P.qpr_magic;
    auto quad_row = [&](int f) { return (int)__umulhi((uint32_t)f, qpr_magic); };
    float4* slot = reinterpret_cast<float4*>(partial) + ((size_t)tile * groups_per_tile + cgroup) * P.slot_quads;
    if (!s_abort) {
        const int f_first = f_begin + (int)threadIdx.x;
        if (cl == 1) {
#pragma unroll 4
            for (int f = f_first; f < f_end; f += blockDim.x) {
                const int row = quad_row(f), cq = f - row * q_per_row;
                const float4 t = *reinterpret_cast<const float4*>(red + row * red_stride + (cq << 2));
                if (direct) store_dw(row, cq, t);
                else slot[f] = t;
            }
        } else {
#pragma unroll 2
            for (int f = f_first; f < f_end; f += blockDim.x) {
                const int row = quad_row(f), cq = f - row * q_per_row;
                const uint32_t src = smem_u32(red + row * red_stride + (cq << 2));
                float4 v[4];                                            // all ranks' pieces first (cl <= 4), then the sum in rank order
#pragma unroll
                for (int rk = 0; rk < 4; ++rk) v[rk] = rk < cl ? ld_dsmem_f4(src, (uint32_t)rk) : make_float4(0.f, 0.f, 0.f, 0.f);
                float4 t = v[0];
#pragma unroll
                for (int rk = 1; rk < 4; ++rk) { t.x += v[rk].x; t.y += v[rk].y; t.z += v[rk].z; t.w += v[rk].w; }
                if (direct) store_dw(row, cq, t);
                else slot[f] = t;
            }
        }
    }
    GACONV_TL(6, threadIdx.x == 0);
    // this CTA no longer reads its peers' blocks: say so now, and wait for the peers' word only before leaving
    if (cl > 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    if (cl > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");      // peers may still be reading this CTA's block
    GACONV_TL(7, threadIdx.x == 0);
#ifdef GACONV_TUNING
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) gaconv_tuning_tc_log[s_log_i][2] = gaconv_globaltimer();
#endif
}

// dYt[n][j][k] = dY[n][k][j] for maps of fewer than 64 pixels (their rows are too short for the copy engine).
// A block takes 64 channels of one image: their maps are one contiguous piece of dY, read in 16-byte units,
// turned in shared memory, and written as pq rows of up to 128 bytes.
__global__ void __launch_bounds__(128)
transpose_dy_kernel(const __nv_bfloat16* __restrict__ dy, __nv_bfloat16* __restrict__ dyt, int k, int pq)
{
    __shared__ __align__(16) unsigned short tile[64 * 32];
    pdl_release_next_grid();
    const int kgroups = (k + 63) / 64;
    const int n = blockIdx.x / kgroups, k0 = (blockIdx.x - n * kgroups) * 64, kg = min(64, k - k0);
    pdl_wait_prior_grid();
    const size_t base = ((size_t)n * k + k0) * pq;                 // first element of map (n, k0); a multiple of 8 elements
    const int elems = kg * pq;
    for (int v = threadIdx.x; v * 8 < elems; v += blockDim.x)
        reinterpret_cast<uint4*>(tile)[v] = __ldg(reinterpret_cast<const uint4*>(dy + base) + v);
    __syncthreads();
    // item = (pixel j, group of eight channels): eight values at stride pq in the tile -> 16 contiguous bytes of dYt
    const int k8 = kg >> 3;
    for (int item = threadIdx.x; item < pq * k8; item += blockDim.x) {
        const int j = item / k8, q = item - j * k8;
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            w[i] = (uint32_t)tile[(8 * q + 2 * i) * pq + j] | ((uint32_t)tile[(8 * q + 2 * i + 1) * pq + j] << 16);
        *reinterpret_cast<uint4*>(dyt + ((size_t)n * pq + j) * k + k0 + 8 * q) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

// Sum of the cluster slots of every tile, for launches whose tiles have many slots: grid (parts, tiles); a CTA
// adds part `blockIdx.x` of tile `blockIdx.y` over the slots -- L lanes per quad, lane l taking slots l, l + L, ...
// in ascending order, eight loads in flight, and a fixed shuffle tree over the lanes -- and writes alpha * sum to dW.
__global__ void __launch_bounds__(256)
reduce_slots_kernel(const float4* __restrict__ partial, float* __restrict__ dw, const TcParams P)
{
    __shared__ int s_coloff[kMaxQuadCols];
    __shared__ signed char s_colvalid[kMaxQuadCols];
    const Geom& g = P.g;
    const int tile = blockIdx.y;
    const int r_lo = P.rsplit ? tile % g.r : 0, kc_tile = P.rsplit ? tile / g.r : tile;
    const int k0 = (kc_tile / P.tiles_c) * P.m, c0 = (kc_tile % P.tiles_c) * P.ct;
    const int nmma = g.s * P.ct, q_per_row = (P.rc * nmma) >> 2;
    pdl_release_next_grid();
    for (int cq = threadIdx.x; cq < q_per_row; cq += blockDim.x) {
        const int col = cq << 2, rl = col / nmma, sc = col - rl * nmma, s_ = sc >> P.ct_shift, c = c0 + (sc & (P.ct - 1));
        s_coloff[cq] = (int)((r_lo + rl) * g.ws_r + s_ * g.ws_s + c * g.ws_c);
        s_colvalid[cq] = (signed char)max(0, min(4, g.c - c));
    }
    __syncthreads();
    pdl_wait_prior_grid();
    const int groups = P.splits / P.cl;
    const int quads = (P.stack ? g.r * P.kb : min(P.m, g.k - k0)) * q_per_row;
    const int part = (quads + (int)gridDim.x - 1) / (int)gridDim.x;
    const int p_begin = min(quads, (int)blockIdx.x * part), npart = min(quads, p_begin + part) - p_begin;
    int lg = 0;
    while (lg < 5 && (2 << lg) * npart <= (int)blockDim.x && (2 << lg) <= groups) ++lg;
    const int L = 1 << lg, sl = threadIdx.x & (L - 1), per_pass = (int)blockDim.x >> lg;
    const float4* slot0 = partial + (size_t)tile * groups * P.slot_quads;
    const bool vec = g.ws_c == 1 && (g.c & 3) == 0;
    for (int base = 0; base < npart; base += per_pass) {
        const int q = base + ((int)threadIdx.x >> lg);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (q < npart) {
            const float4* src = slot0 + p_begin + q;
            for (int gi = sl; gi < groups; gi += 8 * L) {
                float4 u[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) u[j] = gi + j * L < groups ? __ldcg(src + (size_t)(gi + j * L) * P.slot_quads) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int j = 0; j < 8; ++j) { acc.x += u[j].x; acc.y += u[j].y; acc.z += u[j].z; acc.w += u[j].w; }
            }
        }
        for (int off = 1; off < L; off <<= 1) {
            acc.x += __shfl_xor_sync(0xffffffffu, acc.x, off); acc.y += __shfl_xor_sync(0xffffffffu, acc.y, off);
            acc.z += __shfl_xor_sync(0xffffffffu, acc.z, off); acc.w += __shfl_xor_sync(0xffffffffu, acc.w, off);
        }
        if (sl == 0 && q < npart) {
            const int f = p_begin + q, row = (int)__umulhi((uint32_t)f, P.qpr_magic), cq = f - row * q_per_row;
            const int ro = tc_row_offset(P, k0, row);
            if (ro < 0) continue;
            float* p = dw + ro + s_coloff[cq];
            const int valid = s_colvalid[cq];
            const float a = g.alpha;
            if (vec && valid == 4) {
                *reinterpret_cast<float4*>(p) = make_float4(a * acc.x, a * acc.y, a * acc.z, a * acc.w);
            } else {
                const float tv[4] = {acc.x, acc.y, acc.z, acc.w};
                for (int j = 0; j < valid; ++j) p[(size_t)j * g.ws_c] = a * tv[j];
            }
        }
    }
}

// fp32 operand -> two planes: big = x with the 13 low mantissa bits cleared (exactly a TF32 number) and
// small = x - big (exact in fp32; at most 13 significant bits, of which the tensor core keeps 11).  Then
// a*b = big_a*big_b + big_a*small_b + small_a*big_b up to ~2^-21 |a*b|.
__device__ __forceinline__ void split4(const float4 v, float4& b, float4& sm)
{
    b.x = __uint_as_float(__float_as_uint(v.x) & 0xffffe000u); sm.x = v.x - b.x;
    b.y = __uint_as_float(__float_as_uint(v.y) & 0xffffe000u); sm.y = v.y - b.y;
    b.z = __uint_as_float(__float_as_uint(v.z) & 0xffffe000u); sm.z = v.z - b.z;
    b.w = __uint_as_float(__float_as_uint(v.w) & 0xffffe000u); sm.w = v.w - b.w;
}
// one launch for both operands: vectors [0, nx) are X's, [nx, nx + ndy) dY's; planes [big | small] of each
__global__ void __launch_bounds__(256)
split_tf32_kernel(const float4* __restrict__ x, float4* __restrict__ xp, size_t nx,
                  const float4* __restrict__ dy, float4* __restrict__ dyp, size_t ndy)
{
    pdl_release_next_grid();
    pdl_wait_prior_grid();
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < nx + ndy; i += stride) {
        float4 b, sm;
        if (i < nx) { split4(__ldg(x + i), b, sm); xp[i] = b; xp[nx + i] = sm; }
        else { const size_t j = i - nx; split4(__ldg(dy + j), b, sm); dyp[j] = b; dyp[ndy + j] = sm; }
    }
}

// ---------------------------------------------------------------- host side
CUtensorMapSwizzle swizzle_for(int bytes) {
    return bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
}
int swz_code(int bytes) { return bytes == 128 ? 2 : bytes == 64 ? 4 : 6; }
int pow2_ceil(int v) { int p = 32; while (p < v) p *= 2; return p; }
#ifdef GACONV_TUNING
int env_int(const char* name, int dflt) { const char* e = getenv(name); return e ? atoi(e) : dflt; }
#else
constexpr int env_int(const char*, int dflt) { return dflt; }
#endif

// SMs of the current device (one CTA of this kernel fills an SM)
int sm_count()
{
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

// How many clusters of `cl` CTAs of this kernel (one CTA per SM) the current device holds at once.
int resident_clusters(int cl)
{
    static int cached[64][5] = {};
    if (cl <= 1) return sm_count();
    int dev = 0;
    if (cl > 4 || cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return sm_count() / cl * 8 / 10;
    if (cached[dev][cl] == 0) {
        int n = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(1, cl * 64, 1); cfg.blockDim = dim3(256); cfg.dynamicSmemBytes = 200 * 1024;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = cl; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        if (cudaFuncSetAttribute(exact_tc_kernel<0, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024) != cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&n, exact_tc_kernel<0, 0>, &cfg) != cudaSuccess || n < 1) {
            (void)cudaGetLastError();
            n = sm_count() / cl * 8 / 10;          // no answer: a cautious guess
        }
        cached[dev][cl] = n;
    }
    return cached[dev][cl];
}

// Splits of the reduction and cluster size for `tiles` output tiles (fills P.cl, P.splits, P.chunk_base, P.chunk_rem).
bool choose_splits(TcParams& P, const Geom& g, int tiles)
{
    // Splits of the reduction: one wave of CTAs, one per SM.  Consecutive splits form a thread-block cluster of up
    // to 4 that reduces through distributed shared memory; the clusters of a tile meet in the workspace, where the
    // second kernel adds them up.  Larger clusters mean less workspace traffic, but fewer resident CTAs (clusters
    // are placed GPC by GPC: 148 CTAs fit as pairs, 135 as triples, 132 as quadruples).
    // SMs this launch may count on: all of them, or the caller's budget (layers sharing the GPU on several lanes)
    const int sms = g.sm_budget > 0 ? std::min(g.sm_budget, sm_count()) : sm_count();
    int max_splits = env_int("GACONV_TC_SPLITS", 0);
    if (max_splits <= 0) {
        max_splits = sms / tiles;
        if (max_splits < 1) max_splits = 1;
    }
    if (max_splits > P.chunks) max_splits = P.chunks;
    // Sharing the GPU (a budget): no clusters.  The launch is then main-loop-bound on its few SMs, and the cluster
    // barriers and the pull through distributed shared memory cost it more than the workspace pass of the second
    // kernel (measured on the 58-layer step: exact phase 540 -> 526 us).
    const int cl_cap = g.sm_budget > 0 ? 1 : env_int("GACONV_TC_CLUSTER", 4);
    // Measured on the layer shapes of the three networks: a cluster whose splits cover the whole tile (no workspace,
    // no second kernel) wins even at two thirds of the CTAs; otherwise the largest cluster that keeps 85% of them.
    const int cl_force = env_int("GACONV_TC_FORCE_CL", 0);
    int sp_of[5] = {0, 0, 0, 0, 0}, per_of[5] = {0, 0, 0, 0, 0};
    bool fits[5] = {false, false, false, false, false};      // the whole grid is resident at once (no second wave)
    for (int c = 1; c <= 4; ++c) {
        if (c > cl_cap || c > max_splits || (cl_force && c != cl_force)) continue;
        // clusters per tile: within the split budget and, where the tiles allow it, within one resident wave
        const int wave = std::min(resident_clusters(c), std::max(1, sms / c));
        per_of[c] = std::min(max_splits / c, std::max(1, wave / tiles));
        sp_of[c] = per_of[c] * c;
        fits[c] = tiles * per_of[c] <= wave;
    }
    // a cluster size whose grid needs a second wave (a few clusters left over that run alone) is taken only if
    // every size does
    bool any_fit = false;
    for (int c = 1; c <= 4; ++c) any_fit = any_fit || (sp_of[c] > 0 && fits[c]);
    int most = 0;
    for (int c = 1; c <= 4; ++c)
        if (sp_of[c] > 0 && (fits[c] || !any_fit)) most = std::max(most, sp_of[c]);
    int cl = 0, splits = 0;
    // (the shortcut only while a CTA's share of the reduction is short -- up to ~160 k-steps, 128->... at batch 128;
    //  with more work per CTA the idle SMs cost more than the workspace pass: 256->256@8x8 at batch 256, 26 us against 30)
    const long long total_ksteps = (long long)P.chunks * P.ksteps;
    for (int c = 4; c >= 1 && cl == 0; --c)
        if ((fits[c] || !any_fit) && per_of[c] == 1 && sp_of[c] * 10 >= most * 6 &&
            (sp_of[c] == most || g.sm_budget > 0 || total_ksteps <= 160LL * sp_of[c])) {      // (with a budget the other SMs are not idle)
            cl = c; splits = sp_of[c];
        }
    // The tile needs the second kernel anyway.  With a long main loop per CTA (60 k-steps and more) no clusters at
    // all measured faster -- every SM gets a CTA and nobody waits at a cluster barrier (128->128@16x16 20.8 -> 19.6 us,
    // 64->64@32x32 26.4 -> 24.5, 5x5 64->64@16x16 18.7 -> 16.8); with short loops the larger workspace pass loses.
    if (cl == 0 && sp_of[1] == most && (fits[1] || !any_fit) && total_ksteps >= 60LL * most) { cl = 1; splits = sp_of[1]; }
    for (int c = 4; c >= 1 && cl == 0; --c)
        if ((fits[c] || !any_fit) && sp_of[c] > 0 && sp_of[c] * 100 >= most * 85) { cl = c; splits = sp_of[c]; }
    if (cl == 0) return false;
    P.cl = cl;
    P.splits = splits;
    P.reduce_parts = std::max(1, 2 * sms / tiles);          // the second kernel takes the same share of the GPU
    P.chunk_base = P.chunks / splits;
    P.chunk_rem = P.chunks - P.chunk_base * splits;
    return true;
}

}  // namespace

bool plan_tc(const Geom& g, TcPlan* out)
{
    if (!g.bf16) return false;
    if (g.xs_c != 1 || g.c % 8 != 0) return false;                       // NHWC with 16-byte pixel rows
    if (g.stride_h != g.stride_w) return false;
    const int pq = g.p * g.q;
    // maps under 64 pixels: K-major rows of dY would be 32 or 64 bytes (or too short for TMA at all) and the
    // copy engine's cost is per row, so A is taken from a transposed copy with 128-byte rows instead
    const bool tiny = pq < 64 && 64 % pq == 0 && g.k % 8 == 0 && (size_t)g.n * pq >= 64 && env_int("GACONV_TC_TRANSPOSE_SMALL", 1);
    if (!tiny && (pq % 16 != 0 || (pq < 64 && pq != 16 && pq != 32) || (pq >= 64 && pq % 64 != 0))) return false;
    const bool small_map = pq < 64;
    bool halo = !small_map && g.stride_h == 1 && g.q % 8 == 0 && 64 % g.q == 0;
    if (!small_map && !(g.q <= 64 && 64 % g.q == 0)) return false;        // a 64-pixel box must be whole rows
    if (g.r > 7 || g.s > 7) return false;

    TcParams P{};
    P.g = g;
    // M = 64 keeps two accumulators per TMEM column set, which is what lets a 64-channel tile (128-byte
    // rows, the fast MN-major format) hold all three filter rows; M = 128 with 32-channel tiles measured
    // about twice slower per FLOP, so it is used only where the tile is narrow anyway.
    P.m = (g.k <= 64 || g.c >= 64) ? 64 : 128;
    // Many output channels and wide inputs: one filter row per CTA, so that a full-rate M = 128 MMA with a
    // 64-channel (128-byte row) B tile fits tensor memory (S*64 columns) and the epilogue block shrinks.
    // The same split also pays for K <= 64 with 64-channel tiles: the block a CTA has to reduce across its
    // cluster shrinks from 64 x R*S*64 floats (147 KB for 3x3) to a third, and that reduction, not the MMAs,
    // is what a small layer spends its time on.
    P.rsplit = (g.c >= 64 && g.r > 1 && env_int("GACONV_TC_RSPLIT", 1)) ? 1 : 0;
    // Few output channels and narrow inputs (the 16- and 32-channel layers): the MMAs are tiny and the kernel is
    // bound by how fast threads can issue them.  With "same" padding the R filter rows can share ONE MMA: row r
    // of the filter becomes rows r*kb.. of M, fed by the dY box shifted by r image rows (the copy engine fills the
    // rows that leave the map with zeros), against the same X rows.  R times fewer MMAs, and the single
    // accumulator leaves room for the two-issuer scheme.
    const int kb8 = (g.k + 7) / 8 * 8;
    const bool stack = !P.rsplit && !small_map && g.r > 1 && g.r * kb8 <= 128 && g.stride_h == 1 && g.h == g.p &&
                       (g.q % 16 == 0 || g.q == 8) && 64 % g.q == 0 && env_int("GACONV_TC_WIDE", 1) && env_int("GACONV_TC_STACK", 1);
    P.stack = stack ? 1 : 0;
    P.rc = (P.rsplit || stack) ? 1 : g.r;
    if (P.rsplit) P.m = g.k <= 64 ? 64 : 128;
    if (stack) P.m = g.r * kb8 <= 64 ? 64 : 128;
    // One filter row per CTA means one accumulator and one issuing thread, which cannot keep the tensor pipe
    // busy (an MMA of N <= 256 executes in about the time one thread needs to issue it).  So the CTA keeps
    // two accumulators for the row and two issuers take alternate chunks.
    P.dual = (P.rc == 1 && env_int("GACONV_TC_DUAL", 1)) ? 1 : 0;
    P.kb = stack ? kb8 : (g.k < P.m ? (g.k + 7) / 8 * 8 : P.m);
    P.tiny = tiny ? 1 : 0;
    P.kpx = 16; P.passes = 1;
    P.by_image = small_map ? 1 : 0;
    // channels per tile: one swizzle span wide (16, 32 or 64 channels), limited by MMA N <= 256 and TMEM columns
    int ct = g.c >= 64 ? 64 : g.c >= 32 ? 32 : 16;
    const int accs = P.dual ? 2 : P.rc;                 // accumulators of a CTA
    auto cols_for = [&](int c) { return (P.m == 128 ? accs : (accs + 1) / 2) * g.s * c; };
    while (ct > 16 && (g.s * ct > 256 || cols_for(ct) > 512)) ct /= 2;
    if (g.s * ct > 256 || cols_for(ct) > 512) return false;
    if ((g.s * ct) % (P.m == 128 ? 16 : 8) != 0) return false;
    P.ct = ct;
    P.ct_shift = ct == 64 ? 6 : ct == 32 ? 5 : 4;
    P.tiles_k = stack ? 1 : (g.k + P.m - 1) / P.m;
    P.tiles_c = (g.c + ct - 1) / ct;
    if (P.rsplit) halo = false;          // a single row needs no halo rows: its S tiles are loaded directly
    P.halo = halo ? 1 : 0;
    P.a_sub_px = tiny ? 64 : small_map ? pq : 64;      // tiny: 64 reduction rows (images x pixels) per A box
    P.a_swz = swz_code(tiny ? 128 : P.a_sub_px * 2);
    P.b_swz = swz_code(ct * 2);
    // wide tile: stride 1, whole rows per chunk, k-steps inside a row (Q a multiple of 16) or exactly two rows (Q = 8)
    P.wide = (env_int("GACONV_TC_WIDE", 1) && !small_map && g.stride_h == 1 && (g.q % 16 == 0 || g.q == 8) && 64 % g.q == 0) ? 1 : 0;
    // small maps, one filter row per CTA: the (pixel, image) ordering with a single haloed X tile
    const bool tiny2 = tiny && P.rc == 1 && g.stride_h == 1 && g.q % 2 == 0 && g.n >= 8 && env_int("GACONV_TC_TINY2", 1);
    P.tiny2 = tiny2 ? 1 : 0;
    P.b_tiles = (P.wide || tiny2) ? 1 : halo ? g.s : P.rc * g.s;

    // chunk size: as many rows (or images) as fit the stage budget.  The hand-over of a stage costs the producer
    // and the issuer several hundred cycles each, so a stage should carry at least ~8 MMAs.
    // (stacked rows: R copies of every dY box; 66 KB lets a 16-row chunk of the 16- and 32-channel layers fit, three stages)
    const int budget = env_int("GACONV_TC_STAGE_KB", stack ? 66 : 64) * 1024;
    auto stage_bytes = [&](int ci, int bp, int* a_subs, int* tile_bytes, int* tile_stride) {
        const int px = ci * bp * g.q;
        *a_subs = tiny ? px / 64 : small_map ? ci : px / 64;
        const int a_bytes = ((tiny ? (P.m / 64) * px * 128 : small_map ? P.kb * pq * 2 * ci : *a_subs * (stack ? g.r * P.kb : P.kb) * 128) + 1023) / 1024 * 1024;
        const int rows = (halo || P.wide) ? bp + P.rc - 1 : bp;
        *tile_bytes = ci * rows * (P.wide ? g.q + g.s - 1 : g.q) * ct * 2;
        *tile_stride = (*tile_bytes + 1023) / 1024 * 1024;
        return a_bytes + P.b_tiles * *tile_stride;
    };
    int ci = 1, bp = small_map ? g.p : 64 / g.q, a_subs, tb, ts;
    auto tiny2_stage = [&](int c) { return ((P.m / 64) * c * pq * 128 + 1023) / 1024 * 1024 + (g.p * (g.q + g.s - 1) * c * 128 + 1023) / 1024 * 1024; };
    if (tiny2) {
        // reduction rows ordered (pixel, image): a k-step = 16 rows = two pixels x 8 images, one pixel x 16, or half a pixel's 32;
        // as many images per chunk as keep an image row within four k-steps and the stage within the budget
        ci = 8;
        while (ci * 2 <= 32 && g.q * ci * 2 / 16 <= 4 && ci * 2 <= g.n && tiny2_stage(ci * 2) <= budget) ci *= 2;
    } else if (tiny) {
        ci = 64 / pq;                                   // 64 reduction rows = four k-steps per chunk at least
        while (ci * 2 * pq <= 256 && ci * 2 <= g.n && stage_bytes(ci * 2, bp, &a_subs, &tb, &ts) <= budget) ci *= 2;
    } else if (small_map) {
        while (ci * 2 <= 16 && ci * 2 <= g.n && stage_bytes(ci * 2, bp, &a_subs, &tb, &ts) <= budget) ci *= 2;
    } else {
        while (bp * 2 <= g.p && g.p % (bp * 2) == 0 && (halo ? bp * 2 + g.r - 1 : bp * 2 * g.stride_h) <= 256 &&
               stage_bytes(1, bp * 2, &a_subs, &tb, &ts) <= budget) bp *= 2;
        if (g.p % bp != 0) return false;
        // whole maps that are still small: several images per chunk (the wide tile of a single filter row has no
        // halo rows, so the images of a chunk are contiguous in shared memory and the descriptors just keep advancing)
        if (bp == g.p && P.wide && P.rc == 1)
            while (ci * 2 <= 8 && ci * 2 <= g.n && stage_bytes(ci * 2, bp, &a_subs, &tb, &ts) <= budget) ci *= 2;
    }
    P.ci = ci; P.bp = bp;
    P.stage_bytes = stage_bytes(ci, bp, &a_subs, &tb, &ts);
    if (tiny2) {                                        // A: [pixel][image][64 k] per atom; B: [row][column + halo][image][64 c]
        a_subs = g.p;                                   // the issuer walks image rows: Q pixels x ci images = Q * ci / 16 k-steps each
        P.a_sub_px = ci * g.q;
        tb = g.p * (g.q + g.s - 1) * ci * 128;
        ts = (tb + 1023) / 1024 * 1024;
        P.stage_bytes = tiny2_stage(ci);
    }
    P.stage_bytes = (P.stage_bytes + 1023) / 1024 * 1024;
    P.a_subs = a_subs; P.b_tile_bytes = tb; P.b_tile_stride = ts;
    P.a_subs_img = (tiny || small_map) ? a_subs : a_subs / ci;
    P.a_sub_bytes = tiny2 ? ci * g.q * 128 : tiny ? 64 * 128 : small_map ? P.kb * pq * 2 : (stack ? g.r * P.kb : P.kb) * 128;   // small maps: per image; one box carries ci of them
    P.b_lbo = tiny2 ? ci * 128 : P.wide ? ct * 2 : ts;
    P.b_sub_bytes = tiny2 ? (g.q + g.s - 1) * ci * 128 : P.wide ? (P.a_sub_px / g.q) * (g.q + g.s - 1) * ct * 2 : P.a_sub_px * ct * 2;
    P.a_k4_step = tiny ? (16 * 128) >> 4 : 2;
    P.a_lbo = tiny ? ci * pq * 128 : 16;               // tiny: bytes between the 64-channel atoms of an A tile
    P.a_region_bytes = ((tiny ? (P.m / 64) * ci * pq * 128 : P.a_subs * P.a_sub_bytes) + 1023) / 1024 * 1024;
    P.ksteps = ci * bp * g.q / 16;
    P.chunks = (small_map || ci > 1) ? (g.n + ci - 1) / ci : g.n * (g.p / bp);
    const int smem_budget = 200 * 1024;
    P.stages = smem_budget / P.stage_bytes;
    if (P.stages > kMaxStages) P.stages = kMaxStages;
    if (P.stages < 2) return false;
    P.issuers = P.dual ? 2 : P.rc < 3 ? P.rc : 3;
    P.tmem_cols = pow2_ceil(cols_for(ct));
    if (P.tmem_cols > 512) return false;
    // instruction descriptor: fp32 accumulate, bf16 x bf16, A K-major, B MN-major, N, M
    P.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((tiny ? 1u : 0u) << 15) | (1u << 16) | ((uint32_t)(g.s * ct >> 3) << 17) | ((uint32_t)(P.m >> 4) << 24);

    const int tiles = P.tiles_k * P.tiles_c * (P.rsplit ? g.r : 1);
    if (!choose_splits(P, g, tiles)) return false;
    const int splits = P.splits, cl = P.cl;
    // the reduction block must fit the dynamic shared memory (it reuses the operand stages)
    const size_t red_bytes = (size_t)P.m * (P.rc * g.s * ct + 4) * 4;
    if (red_bytes > 212 * 1024) return false;
        P.slot_quads = P.m * (P.rc * g.s * ct / 4);
    P.qpr_magic = (uint32_t)(((1ull << 32) + (P.rc * g.s * ct / 4) - 1) / (P.rc * g.s * ct / 4));
    P.timeline = env_int("GACONV_TC_TIMELINE", 0);
#ifdef GACONV_TUNING
    if (env_int("GACONV_TC_VERBOSE", 0))
        fprintf(stderr, "plan_tc c%d k%d pq%d: m%d ct%d rsplit%d dual%d wide%d tiny%d/%d ci%d bp%d ksteps%d stage %d B x%d, tiles %d splits %d cl %d chunks %d\n",
                g.c, g.k, pq, P.m, ct, P.rsplit, P.dual, P.wide, P.tiny, P.tiny2, ci, bp, P.ksteps, P.stage_bytes, P.stages, tiles, splits, cl, P.chunks);
#endif

    out->partial_bytes = splits / cl > 1 ? (size_t)tiles * (splits / cl) * P.slot_quads * 16 : 0;
    out->scratch_bytes = tiny ? (size_t)g.n * g.k * pq * 2 : 0;      // transposed copy of dY
    out->reads_transposed_dy = tiny;
    out->stacked_rows = P.stack != 0;
    static_assert(sizeof(TcParams) <= sizeof(out->opaque), "TcPlan::opaque too small");
    memcpy(out->opaque, &P, sizeof(P));
    return encode_fn() != nullptr;
}

// fp32 inputs on the tcgen05 path (kind::tf32): single-row CTAs with the wide X tile, stride 1, rows of 8, 16 or 32
// output pixels.  passes = 3 (fp32 accuracy through split operands) or 1 (plain TF32).
bool plan_tc_f32(const Geom& g, int passes, TcPlan* out)
{
    if (g.bf16 || g.xs_c != 1 || g.c % 32 != 0) return false;
    if (g.stride_h != 1 || g.stride_w != 1 || g.r > 7 || g.s > 7 || g.s * 32 > 256) return false;
    const int pq = g.p * g.q;
    if (pq % 32 != 0 || g.q % 8 != 0 || 32 % g.q != 0) return false;          // a 32-pixel box is whole rows, a k-step lies in a row
    if ((size_t)g.n * g.c * g.h * g.w % 4 != 0 || (size_t)g.n * g.k * pq % 4 != 0) return false;
    TcParams P{};
    P.g = g;
    P.f32 = 1; P.passes = passes; P.kpx = 8;
    P.m = g.k <= 64 ? 64 : 128;
    // few output channels and "same" padding: all filter rows stacked in M, as in the bf16 plan
    const int kb8 = (g.k + 7) / 8 * 8;
    const bool stack = g.r > 1 && g.r * kb8 <= 128 && g.h == g.p && env_int("GACONV_TC_STACK", 1);
    P.stack = stack ? 1 : 0;
    if (stack) P.m = g.r * kb8 <= 64 ? 64 : 128;
    P.rsplit = (!stack && g.r > 1) ? 1 : 0;
    P.rc = 1; P.dual = 1; P.issuers = 2;
    P.kb = stack ? kb8 : (g.k < P.m ? (g.k + 7) / 8 * 8 : P.m);
    const int arows = stack ? g.r * kb8 : P.kb;          // rows of a dY sub-tile (32 pixels) in shared memory
    const int ct = 32;
    P.ct = ct; P.ct_shift = 5;
    P.tiles_k = stack ? 1 : (g.k + P.m - 1) / P.m;
    P.tiles_c = (g.c + ct - 1) / ct;
    P.wide = 1; P.b_tiles = 1;
    P.a_sub_px = 32;
    P.a_swz = swz_code(128); P.b_swz = 1;               // B: 128-byte swizzle with 32-byte base (MN-major 32-bit elements)
    const int planes = passes == 3 ? 2 : 1;
    const int budget = env_int("GACONV_TC_STAGE_KB", stack ? 66 : 64) * 1024, wt = g.q + g.s - 1;
    auto stage = [&](int ci, int bp, int* a_bytes, int* tile_bytes) {
        *a_bytes = (ci * bp * g.q / 32 * arows * 128 + 1023) / 1024 * 1024;
        *tile_bytes = (ci * bp * wt * ct * 4 + 1023) / 1024 * 1024;
        return planes * (*a_bytes + *tile_bytes);
    };
    int ci = 1, bp = 32 / g.q, ab, tb;
    while (bp * 2 <= g.p && g.p % (bp * 2) == 0 && bp * 2 <= 256 && stage(1, bp * 2, &ab, &tb) <= budget) bp *= 2;
    if (g.p % bp != 0) return false;
    if (bp == g.p)
        while (ci * 2 <= 8 && ci * 2 <= g.n && stage(ci * 2, bp, &ab, &tb) <= budget) ci *= 2;
    P.ci = ci; P.bp = bp;
    P.stage_bytes = stage(ci, bp, &ab, &tb);
    P.a_subs = ci * bp * g.q / 32;
    P.a_subs_img = P.a_subs / ci;
    P.a_sub_bytes = arows * 128;
    P.a_k4_step = 2;                                    // eight fp32 pixels = 32 bytes
    P.a_lbo = 16;
    P.a_region_bytes = planes * ab;
    P.a_plane_bytes = ab; P.b_plane_bytes = tb;
    P.b_tile_bytes = ci * bp * wt * ct * 4; P.b_tile_stride = tb;
    P.b_lbo = ct * 4;                                   // a column shift = one pixel = 128 bytes
    P.b_sub_bytes = (32 / g.q) * wt * ct * 4;
    P.ksteps = ci * bp * g.q / 8;
    P.chunks = ci > 1 ? (g.n + ci - 1) / ci : g.n * (g.p / bp);
    P.stages = 200 * 1024 / P.stage_bytes;
    if (P.stages > kMaxStages) P.stages = kMaxStages;
    if (P.stages < 2) return false;
    const int cols = (P.m == 128 ? 2 : 1) * g.s * ct;   // two accumulators: side by side (M = 128) or in the lane halves (M = 64)
    if ((g.s * ct) % (P.m == 128 ? 16 : 8) != 0) return false;
    P.tmem_cols = pow2_ceil(cols);
    if (P.tmem_cols > 512) return false;
    // instruction descriptor: fp32 accumulate, tf32 x tf32, A K-major, B MN-major, N, M
    P.idesc = (1u << 4) | (2u << 7) | (2u << 10) | (1u << 16) | ((uint32_t)(g.s * ct >> 3) << 17) | ((uint32_t)(P.m >> 4) << 24);
    const int tiles = P.tiles_k * P.tiles_c * (P.rsplit ? g.r : 1);
    if (!choose_splits(P, g, tiles)) return false;
    if ((size_t)P.m * (g.s * ct + 4) * 4 > 212 * 1024) return false;
    P.slot_quads = P.m * (g.s * ct / 4);
    P.qpr_magic = (uint32_t)(((1ull << 32) + (g.s * ct / 4) - 1) / (g.s * ct / 4));
    P.timeline = env_int("GACONV_TC_TIMELINE", 0);
#ifdef GACONV_TUNING
    if (env_int("GACONV_TC_VERBOSE", 0))
        fprintf(stderr, "plan_tc_f32 c%d k%d pq%d passes%d: m%d ci%d bp%d ksteps%d stage %d B x%d, tiles %d splits %d cl %d chunks %d\n",
                g.c, g.k, pq, passes, P.m, ci, bp, P.ksteps, P.stage_bytes, P.stages, tiles, P.splits, P.cl, P.chunks);
#endif
    out->partial_bytes = P.splits / P.cl > 1 ? (size_t)tiles * (P.splits / P.cl) * P.slot_quads * 16 : 0;
    // the two planes of each operand, [plane][elements]
    out->scratch_bytes = passes == 3 ? 2 * ((size_t)g.n * g.c * g.h * g.w + (size_t)g.n * g.k * pq) * 4 : 0;
    out->reads_transposed_dy = false;
    out->stacked_rows = P.stack != 0;
    memcpy(out->opaque, &P, sizeof(P));
    return encode_fn() != nullptr;
}

cudaError_t launch_tc(const void* x, const void* dy, float* dw, float* partial, void* scratch, uint32_t* counters,
                      uint32_t* status, const TcPlan& plan, cudaStream_t stream)
{
    TcParams P;
    memcpy(&P, plan.opaque, sizeof(P));
    const Geom& g = P.g;
    const int pq = g.p * g.q;
    EncodeTiledFn enc = encode_fn();
    if (enc == nullptr) return cudaErrorNotSupported;

    CUtensorMap map_dy, map_x;
    if (P.f32) {
        const size_t nx = (size_t)g.n * g.c * g.h * g.w, ndy = (size_t)g.n * g.k * pq;
        const void* xs = x; const void* dys = dy;
        if (P.passes == 3) {      // planes [big | small] of X, then of dY, in the scratch
            float* xp = static_cast<float*>(scratch); float* dyp = xp + 2 * nx;
            const unsigned blocks = 148 * 8;
            if (launch_kernel(split_tf32_kernel, dim3(blocks), dim3(256), 0, stream, dim3(1, 1, 1), static_cast<const float4*>(x),
                              reinterpret_cast<float4*>(xp), nx / 4, static_cast<const float4*>(dy), reinterpret_cast<float4*>(dyp), ndy / 4) != cudaSuccess)
                return cudaErrorLaunchFailure;
            note_launch();
            xs = xp; dys = dyp;
        }
        const cuuint64_t planes = P.passes == 3 ? 2 : 1;
        cuuint64_t d4[4] = {(cuuint64_t)pq, (cuuint64_t)g.k, (cuuint64_t)g.n, planes};
        cuuint64_t s4[3] = {(cuuint64_t)pq * 4, (cuuint64_t)g.k * pq * 4, (cuuint64_t)ndy * 4};
        cuuint32_t b4[4] = {32, (cuuint32_t)P.kb, 1, 1}, e4[4] = {1, 1, 1, 1};
        cuuint64_t d5[5] = {(cuuint64_t)g.c, (cuuint64_t)g.w, (cuuint64_t)g.h, (cuuint64_t)g.n, planes};
        cuuint64_t s5[4] = {(cuuint64_t)g.c * 4, (cuuint64_t)g.w * g.c * 4, (cuuint64_t)g.h * g.w * g.c * 4, (cuuint64_t)nx * 4};
        cuuint32_t b5[5] = {(cuuint32_t)P.ct, (cuuint32_t)(g.q + g.s - 1), (cuuint32_t)P.bp, (cuuint32_t)P.ci, 1}, e5[5] = {1, 1, 1, 1, 1};
        if (enc(&map_dy, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<void*>(dys), d4, s4, b4, e4, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
            enc(&map_x, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5, const_cast<void*>(xs), d5, s5, b5, e5, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    } else if (P.tiny) {   // transposed copy dYt[n][pq][k], then a map over (k, pq, n) -- (k, n, pq) for the (pixel, image) ordering -- with 64-channel boxes
        if (dy != nullptr) {
            if (launch_kernel(transpose_dy_kernel, dim3((unsigned)(g.n * ((g.k + 63) / 64))), dim3(128), 0, stream, dim3(1, 1, 1),
                              static_cast<const __nv_bfloat16*>(dy), static_cast<__nv_bfloat16*>(scratch), g.k, pq) != cudaSuccess)
                return cudaErrorLaunchFailure;
            note_launch();
        }
        cuuint64_t dims[3] = {(cuuint64_t)g.k, (cuuint64_t)pq, (cuuint64_t)g.n};
        cuuint64_t strides[2] = {(cuuint64_t)g.k * 2, (cuuint64_t)g.k * pq * 2};
        cuuint32_t box[3] = {64, (cuuint32_t)pq, (cuuint32_t)P.ci};
        cuuint32_t es[3] = {1, 1, 1};
        if (P.tiny2) {      // the same array seen as (k, n, pq): a box lands as [pixel][image][k]
            dims[1] = (cuuint64_t)g.n; dims[2] = (cuuint64_t)pq;
            strides[0] = (cuuint64_t)g.k * pq * 2; strides[1] = (cuuint64_t)g.k * 2;
            box[1] = (cuuint32_t)P.ci; box[2] = (cuuint32_t)pq;
        }
        if (enc(&map_dy, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, scratch, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    } else {   // dY as (pq, k, n), bf16
        cuuint64_t dims[3] = {(cuuint64_t)pq, (cuuint64_t)g.k, (cuuint64_t)g.n};
        cuuint64_t strides[2] = {(cuuint64_t)pq * 2, (cuuint64_t)g.k * pq * 2};
        cuuint32_t box[3] = {(cuuint32_t)P.a_sub_px, (cuuint32_t)P.kb, (cuuint32_t)(P.a_sub_px < 64 ? P.ci : 1)};
        cuuint32_t es[3] = {1, 1, 1};
        if (enc(&map_dy, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(dy), dims, strides, box, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(P.a_sub_px * 2), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    if (!P.f32) {   // X as (c, w, h, n), bf16; a box is ct channels x q columns x rows x ci images, stepping by the conv stride
        cuuint64_t dims[4] = {(cuuint64_t)g.c, (cuuint64_t)g.w, (cuuint64_t)g.h, (cuuint64_t)g.n};
        cuuint64_t strides[3] = {(cuuint64_t)g.c * 2, (cuuint64_t)g.w * g.c * 2, (cuuint64_t)g.h * g.w * g.c * 2};
        const int rows = (P.halo || P.wide) ? P.bp + P.rc - 1 : P.bp;
        const int cols = P.wide ? g.q + g.s - 1 : g.q * g.stride_w;
        cuuint32_t box[4] = {(cuuint32_t)P.ct, (cuuint32_t)cols, (cuuint32_t)(rows * g.stride_h), (cuuint32_t)P.ci};
        cuuint32_t es[4] = {1, (cuuint32_t)g.stride_w, (cuuint32_t)g.stride_h, 1};
        if (P.tiny2) {      // X seen as (c, n, w, h): a box of P rows x (Q + S - 1) columns x ci images lands as [row][column][image][c]
            dims[1] = (cuuint64_t)g.n; dims[2] = (cuuint64_t)g.w; dims[3] = (cuuint64_t)g.h;
            strides[0] = (cuuint64_t)g.h * g.w * g.c * 2; strides[1] = (cuuint64_t)g.c * 2; strides[2] = (cuuint64_t)g.w * g.c * 2;
            box[1] = (cuuint32_t)P.ci; box[2] = (cuuint32_t)(g.q + g.s - 1); box[3] = (cuuint32_t)g.p;
            es[1] = es[2] = es[3] = 1;
        }
        if (enc(&map_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(x), dims, strides, box, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(P.ct * 2), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    // dynamic shared memory: stages, 1 KiB of alignment slack, and a tail so that the MMA's read of
    // all M rows of an A box with fewer valid rows stays inside the allocation
    size_t smem = (size_t)P.stages * P.stage_bytes;
    const size_t red_bytes = (size_t)P.m * (P.rc * g.s * P.ct + 4) * 4;
    if (red_bytes > smem) smem = red_bytes;
    smem += 1024 + (size_t)P.m * 128;
    dim3 grid(P.tiles_k * P.tiles_c * (P.rsplit ? g.r : 1), P.splits);
    const int ks = P.a_sub_px / (P.f32 ? 8 : 16);
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) dev = -1;
    cudaError_t err = cudaErrorInvalidValue;
#define GACONV_TC_CASE(RR, KK)                                                                                     \
    if (err == cudaErrorInvalidValue && (RR == 0 || (P.rc == RR && ks == KK))) {                                     \
        static size_t configured[64] = {};           /* the attribute is per device */                            \
        err = cudaSuccess;                                                                                         \
        if (dev < 0 || dev >= 64 || smem > configured[dev]) {                                                      \
            err = cudaFuncSetAttribute(exact_tc_kernel<RR, KK>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
            if (err == cudaSuccess && dev >= 0 && dev < 64) configured[dev] = smem;                                \
        }                                                                                                          \
        if (err == cudaSuccess) {                                                                                  \
            err = launch_kernel(exact_tc_kernel<RR, KK>, grid, dim3(256), smem, stream, dim3(1, P.cl, 1), map_dy, map_x, dw, \
                                partial, counters, status, P);                                                    \
        }                                                                                                          \
    }
    GACONV_TC_CASE(3, 4)
    GACONV_TC_CASE(3, 1)
    GACONV_TC_CASE(5, 4)
    GACONV_TC_CASE(1, 4)
    GACONV_TC_CASE(1, 2)
    GACONV_TC_CASE(1, 1)
    GACONV_TC_CASE(0, 0)
#undef GACONV_TC_CASE
    if (err != cudaSuccess) return err;
    note_launch();
    if (P.splits / P.cl > 1) {
        err = launch_kernel(reduce_slots_kernel, dim3(P.reduce_parts, grid.x), dim3(256), 0, stream, dim3(1, 1, 1),
                            reinterpret_cast<const float4*>(partial), dw, P);
        if (err != cudaSuccess) return err;
        note_launch();
    }
    return cudaGetLastError();
}

}  // namespace gaconv

#ifdef GACONV_TUNING
// tuning builds: global-timer stamps (ns) of every CTA of the last tensor-core launch, [1024][8]
extern "C" int gaconv_tuning_read_stamps(unsigned long long* host)
{
    return (int)cudaMemcpyFromSymbol(host, gaconv_tuning_stamps, sizeof(gaconv_tuning_stamps));
}
extern "C" int gaconv_tuning_read_tc_log(unsigned long long* host, unsigned int* count)
{
    if (cudaMemcpyFromSymbol(count, gaconv_tuning_tc_log_n, sizeof(unsigned int)) != cudaSuccess) return 1;
    return (int)cudaMemcpyFromSymbol(host, gaconv_tuning_tc_log, sizeof(gaconv_tuning_tc_log));
}
#endif
