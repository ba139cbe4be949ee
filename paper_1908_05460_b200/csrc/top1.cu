// Max-gradient approximation (paper Section 2.3, Algorithm 1).  top1_fused_kernel does the whole method
// in one launch (thread-block clusters, distributed shared memory); the two-kernel form below is kept
// for shapes whose per-channel block does not fit shared memory and for the inspection entry point:
//   select_kernel  -- per (n,k) map of dY: position of the largest magnitude (lowest index among
//                     equals) and the signed sum of the map      [Algorithm 1, arg-max and sum lines]
//   gather_kernel  -- dW[k,r,s,c] = alpha * sum_n sum[n,k] * Xz[n, c, patch at the selected position]
//                                                                  [Algorithm 1, accumulation line]
// The top-k variant (Section 2.3, last sentence) selects with select_topk_kernel and feeds the list to
// top1_fused_kernel (k records per image), or to gather_kernel when the records do not fit shared memory;
// select_sparse_transposed_kernel writes the sparse tensor the dense route contracts on small maps.
// Selection compares the bit pattern of |v| in the input dtype as an unsigned integer, which orders
// finite values exactly as their magnitudes do (NaN above Inf), so indices are reproducible bit for bit.
#include <cooperative_groups.h>

#include "gaconv_internal.h"
#include "device_utils.cuh"

namespace gaconv {

namespace {

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }

// ---- per-element visitor: track (largest |bits|, first index) and the running sum ----
struct Scan {
    int best_mag;   // -1 before the first element so that any element replaces it
    int best_j;
    float sum;
    __device__ __forceinline__ void take(uint32_t mag, int j, float v) {
        if ((int)mag > best_mag) { best_mag = (int)mag; best_j = j; }
        sum += v;
    }
};

template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int kPerVec = 4;
    __device__ static __forceinline__ void visit(const uint4& v, int j0, Scan& sc) {
        sc.take(v.x & 0x7fffffffu, j0 + 0, __uint_as_float(v.x));
        sc.take(v.y & 0x7fffffffu, j0 + 1, __uint_as_float(v.y));
        sc.take(v.z & 0x7fffffffu, j0 + 2, __uint_as_float(v.z));
        sc.take(v.w & 0x7fffffffu, j0 + 3, __uint_as_float(v.w));
    }
    __device__ static __forceinline__ void visit1(const float* p, int j, Scan& sc) {
        uint32_t b = __float_as_uint(p[j]);
        sc.take(b & 0x7fffffffu, j, __uint_as_float(b));
    }
    __device__ static __forceinline__ float round_to_T(float v) { return v; }
    __device__ static __forceinline__ void store1(float* p, float v) { *p = v; }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kPerVec = 8;
    __device__ static __forceinline__ void visit(const uint4& v, int j0, Scan& sc) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t lo = w[i] & 0xffffu, hi = w[i] >> 16;
            sc.take(lo & 0x7fffu, j0 + 2 * i, bf16_bits_to_float(lo));
            sc.take(hi & 0x7fffu, j0 + 2 * i + 1, bf16_bits_to_float(hi));
        }
    }
    __device__ static __forceinline__ void visit1(const __nv_bfloat16* p, int j, Scan& sc) {
        uint32_t b = *reinterpret_cast<const unsigned short*>(p + j);
        sc.take(b & 0x7fffu, j, bf16_bits_to_float(b));
    }
    __device__ static __forceinline__ void store1(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
};

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// A group of G lanes (G a power of two, G <= 32) scans one map: each lane takes every G-th 16-byte
// vector (VEC: maps are a whole number of vectors, hence 16-byte aligned) or every G-th element, keeps
// its first largest magnitude and its running sum; the lanes are then combined -- larger magnitude
// wins, then the lower index; sums add in a fixed tree.  All 32 lanes of the warp must call this.
template <typename T, bool VEC>
__device__ __forceinline__ void scan_map(const T* __restrict__ map, bool live, int pq, int G, int sub,
                                         int& best_j, float& sum)
{
    Scan sc{-1, 0, 0.0f};
    if (live) {
        if (VEC) {
            constexpr int E = Elem<T>::kPerVec;
            const uint4* mv = reinterpret_cast<const uint4*>(map);
            const int nvec = pq / E;
            int v = sub;
            // eight, then four independent loads in flight per lane before any is consumed
            for (; v + 7 * G < nvec; v += 8 * G) {
                uint4 a[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) a[u] = ld_stream(mv + v + u * G);
#pragma unroll
                for (int u = 0; u < 8; ++u) Elem<T>::visit(a[u], (v + u * G) * E, sc);
            }
            for (; v + 3 * G < nvec; v += 4 * G) {
                uint4 a = ld_stream(mv + v), b = ld_stream(mv + v + G), c = ld_stream(mv + v + 2 * G),
                      d = ld_stream(mv + v + 3 * G);
                Elem<T>::visit(a, v * E, sc);
                Elem<T>::visit(b, (v + G) * E, sc);
                Elem<T>::visit(c, (v + 2 * G) * E, sc);
                Elem<T>::visit(d, (v + 3 * G) * E, sc);
            }
            for (; v < nvec; v += G) { uint4 a = ld_stream(mv + v); Elem<T>::visit(a, v * E, sc); }
        } else {
            for (int j = sub; j < pq; j += G) Elem<T>::visit1(map, j, sc);
        }
    }
    unsigned long long key = ((unsigned long long)(unsigned)(sc.best_mag + 1) << 32) | (0xffffffffu - (unsigned)sc.best_j);
    float s = sc.sum;
    for (int off = G >> 1; off > 0; off >>= 1) {
        unsigned long long other = __shfl_xor_sync(0xffffffffu, key, off);
        float so = __shfl_xor_sync(0xffffffffu, s, off);
        key = other > key ? other : key;
        s += so;
    }
    best_j = (int)(0xffffffffu - (unsigned)(key & 0xffffffffu));
    sum = s;
}

// Selection alone (inspection entry point): idx, sum and optionally the dense sparse tensor.
template <typename T, bool VEC>
__global__ void __launch_bounds__(256)
select_kernel(const T* __restrict__ dy, int32_t* __restrict__ idx, float* __restrict__ sum,
              T* __restrict__ dy_sparse, long long num_maps, int pq, int G)
{
    pdl_release_next_grid();
    pdl_wait_prior_grid();
    const int lane = threadIdx.x & 31;
    const int sub = lane & (G - 1);
    const long long warp = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long long m = warp * (32 / G) + lane / G;
    const bool live = m < num_maps;
    int best_j; float s;
    scan_map<T, VEC>(dy + (live ? m : 0) * (long long)pq, live, pq, G, sub, best_j, s);
    if (!live) return;
    if (sub == 0) { idx[m] = best_j; sum[m] = s; }
    if (dy_sparse != nullptr) {
        T* out = dy_sparse + m * (long long)pq;
        if (VEC) {      // 16-byte zero vectors, then the one retained entry
            constexpr int E = Elem<T>::kPerVec;
            uint4* ov = reinterpret_cast<uint4*>(out);
            for (int v = sub; v < pq / E; v += G) ov[v] = make_uint4(0u, 0u, 0u, 0u);
            __syncwarp();
            if (sub == 0) Elem<T>::store1(out + best_j, s);
        } else {
            for (int j = sub; j < pq; j += G) Elem<T>::store1(out + j, j == best_j ? s : 0.0f);
        }
    }
}

// Selection for the route "sparse dY + dense tensor-core kernel" on maps of fewer than 64 pixels, where that kernel
// reads a transposed copy dYt[n][j][k] of its dY operand: writes the sparse tensor straight in that layout (the
// signed sum, rounded to bf16, at the retained position of every map, zero elsewhere).  A block takes 64 channels
// of one image: one thread per map scans its pq <= 32 elements, then the block writes pq rows of up to 128 bytes.
__global__ void __launch_bounds__(128)
select_sparse_transposed_kernel(const __nv_bfloat16* __restrict__ dy, __nv_bfloat16* __restrict__ dyt, int k, int pq)
{
    __shared__ int s_idx[64];
    __shared__ unsigned short s_val[64];
    pdl_release_next_grid();
    const int kgroups = (k + 63) / 64;
    const int n = blockIdx.x / kgroups, k0 = (blockIdx.x - n * kgroups) * 64, kg = min(64, k - k0);
    pdl_wait_prior_grid();
    if ((int)threadIdx.x < kg) {
        const __nv_bfloat16* map = dy + ((size_t)n * k + k0 + threadIdx.x) * pq;
        Scan sc{-1, 0, 0.0f};
        for (int j = 0; j < pq; ++j) Elem<__nv_bfloat16>::visit1(map, j, sc);
        s_idx[threadIdx.x] = sc.best_j;
        s_val[threadIdx.x] = __bfloat16_as_ushort(__float2bfloat16_rn(sc.sum));
    }
    __syncthreads();
    const int k8 = kg >> 3;
    for (int item = threadIdx.x; item < pq * k8; item += blockDim.x) {
        const int j = item / k8, q = item - j * k8;
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t lo = s_idx[8 * q + 2 * i] == j ? s_val[8 * q + 2 * i] : 0u;
            const uint32_t hi = s_idx[8 * q + 2 * i + 1] == j ? s_val[8 * q + 2 * i + 1] : 0u;
            w[i] = lo | (hi << 16);
        }
        *reinterpret_cast<uint4*>(dyt + ((size_t)n * pq + j) * k + k0 + 8 * q) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

// Selection of the top-k variant: one warp per map.  Round t picks the largest key below the key picked in
// round t-1, where key = (bit pattern of |v|, complement of the position): keys are distinct, larger magnitude
// first and, among equal magnitudes, the lower position first -- the order the single arg-max uses.
template <typename T>
__global__ void __launch_bounds__(256)
select_topk_kernel(const T* __restrict__ dy, int32_t* __restrict__ idx, float* __restrict__ sum, long long num_maps, int pq, int topk)
{
    pdl_release_next_grid();
    pdl_wait_prior_grid();
    const int lane = threadIdx.x & 31;
    const long long m = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (m >= num_maps) return;
    const T* map = dy + m * (long long)pq;
    unsigned long long prev = ~0ull;
    float total = 0.0f;
    for (int t = 0; t < topk; ++t) {
        unsigned long long best = 0ull;
        for (int j = lane; j < pq; j += 32) {
            Scan sc{-1, 0, 0.0f};
            Elem<T>::visit1(map, j, sc);
            const unsigned long long key = ((unsigned long long)(unsigned)(sc.best_mag + 1) << 32) | (0xffffffffu - (unsigned)j);
            if (key < prev && key > best) best = key;
            if (t == 0) total += sc.sum;
        }
        for (int off = 16; off > 0; off >>= 1) {
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, off);
            best = other > best ? other : best;
        }
        if (lane == 0) idx[m * topk + t] = (int)(0xffffffffu - (unsigned)(best & 0xffffffffu));
        prev = best;
    }
    for (int off = 16; off > 0; off >>= 1) total += __shfl_xor_sync(0xffffffffu, total, off);
    if (lane == 0) sum[m] = total;
}

// four consecutive elements, raw (16-byte load for fp32, 8-byte load for bf16), and their values as floats
struct Raw4 { uint32_t w[4]; };
__device__ __forceinline__ Raw4 ld4_raw(const float* p) {
    const uint4 t = __ldg(reinterpret_cast<const uint4*>(p));
    return Raw4{{t.x, t.y, t.z, t.w}};
}
__device__ __forceinline__ Raw4 ld4_raw(const __nv_bfloat16* p) {
    const uint2 t = __ldg(reinterpret_cast<const uint2*>(p));
    return Raw4{{t.x, t.y, 0u, 0u}};
}
__device__ __forceinline__ Raw4 ld8_raw(const __nv_bfloat16* p) {          // eight channels
    const uint4 t = __ldg(reinterpret_cast<const uint4*>(p));
    return Raw4{{t.x, t.y, t.z, t.w}};
}
__device__ __forceinline__ Raw4 ld8_raw(const float* p) { return ld4_raw(p); }   // (never used: fp32 loads are 16 bytes already)
__device__ __forceinline__ void raw_to_float8(const Raw4& r, float (&v)[8]) {
#pragma unroll
    for (int i = 0; i < 4; ++i) { v[2 * i] = __uint_as_float(r.w[i] << 16); v[2 * i + 1] = __uint_as_float(r.w[i] & 0xffff0000u); }
}
__device__ __forceinline__ void raw_to_float(const Raw4& r, const float*, float (&v)[4]) {
    v[0] = __uint_as_float(r.w[0]); v[1] = __uint_as_float(r.w[1]); v[2] = __uint_as_float(r.w[2]); v[3] = __uint_as_float(r.w[3]);
}
__device__ __forceinline__ void raw_to_float(const Raw4& r, const __nv_bfloat16*, float (&v)[4]) {
    v[0] = __uint_as_float(r.w[0] << 16); v[1] = __uint_as_float(r.w[0] & 0xffff0000u);
    v[2] = __uint_as_float(r.w[1] << 16); v[3] = __uint_as_float(r.w[1] & 0xffff0000u);
}

// Algorithm 1 in one launch.  grid (CL, K), thread-block clusters of CL CTAs along x: the CL CTAs of
// a cluster share one output channel k and split the batch into CL contiguous ranges of images.
//   phase 1  each CTA scans the dY maps of its images (selection),
//   phase 2  accumulates their patches, images in order, into a shared-memory block of R*S*C sums,
//   phase 3  after a cluster barrier, CTA j adds slice j of the block over the CL CTAs through
//            distributed shared memory, in rank order, and writes alpha * total to dW.
// No global scratch, no atomics; the order of every sum is fixed.
#ifdef GACONV_TUNING
// tuning builds: CTA (0,0) of every launch logs {entry, dependency satisfied, exit} in nanoseconds
__device__ unsigned long long gaconv_tuning_top1_log[4096][4];
__device__ unsigned int gaconv_tuning_top1_log_n;
__device__ __forceinline__ unsigned long long tuning_now() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
#endif

template <typename T, bool VEC, bool WIDE>
__global__ void __launch_bounds__(512, 2)
top1_fused_kernel(const T* __restrict__ x, const T* __restrict__ dy, float* __restrict__ dw, Geom g, int ipc, int G, bool vec_x, int NJ,
                  const int32_t* __restrict__ sel_idx, const float* __restrict__ sel_sum, int topk)
{
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
#ifdef GACONV_TUNING
    const unsigned long long t_in = tuning_now();
    const bool logger = blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0;
    unsigned int log_i = 0;
#endif
    pdl_wait_prior_grid();
#ifdef GACONV_TUNING
    if (logger) {
        log_i = atomicAdd(&gaconv_tuning_top1_log_n, 1u) & 4095u;
        gaconv_tuning_top1_log[log_i][0] = t_in; gaconv_tuning_top1_log[log_i][1] = tuning_now();
        gaconv_tuning_top1_log[log_i][3] = ((unsigned long long)g.c << 32) | (unsigned)(g.k * 65536 + g.p);
    }
#endif
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int rsc = g.r * g.s * g.c;
    float* s_part = reinterpret_cast<float*>(smem_raw);                 // [rsc]
    // per image of this CTA, one 16-byte record: {element offset of the patch's top-left pixel (64 bits), the signed
    // sum (float bits), validity bits: bit r = patch row r lies inside the image, bit 16+s = patch column s does}
    uint4* s_rec = reinterpret_cast<uint4*>(smem_raw + (((size_t)rsc * 4 + 15) & ~(size_t)15));      // [ipc]
    float* s_subs = reinterpret_cast<float*>(s_rec + ipc * topk);       // [NJ][rsc] lane subtotals

    const int k = blockIdx.y, chunk = blockIdx.x, CL = gridDim.x;
    const int n0 = chunk * ipc;
    const int cnt = max(0, min(ipc, g.n - n0));
    const int pq = g.p * g.q;

    // ---- phase 1: selection (or, for the top-k method, the list another kernel selected) ----
    auto put_record = [&](int slot, int i, int j, float weight) {
        const int h0 = (j / g.q) * g.stride_h - g.pad_h, w0 = (j % g.q) * g.stride_w - g.pad_w;
        const long long base = (long long)i * g.xs_n + (long long)h0 * g.xs_h + (long long)w0 * g.xs_w;
        uint32_t mask = 0;
        for (int r = 0; r < g.r; ++r) mask |= (uint32_t)((unsigned)(h0 + r) < (unsigned)g.h) << r;
        for (int c = 0; c < g.s; ++c) mask |= (uint32_t)((unsigned)(w0 + c) < (unsigned)g.w) << (16 + c);
        s_rec[slot] = make_uint4((uint32_t)(unsigned long long)base, (uint32_t)((unsigned long long)base >> 32), __float_as_uint(weight), mask);
    };
    if (sel_idx != nullptr) {
        // record (image i, entry t): the retained position with weight sum / topk; images in order, entries in order of selection
        for (int e = threadIdx.x; e < cnt * topk; e += blockDim.x) {
            const int i = e / topk;
            const long long m = (long long)(n0 + i) * g.k + k;
            put_record(e, i, sel_idx[m * topk + (e - i * topk)], sel_sum[m] / (float)topk);
        }
    } else {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        const int sub = lane & (G - 1), per_warp = 32 / G, per_pass = (blockDim.x >> 5) * per_warp;
        for (int base = 0; base < cnt; base += per_pass) {
            const int i = base + warp * per_warp + lane / G;
            const bool live = i < cnt;
            int best_j; float s;
            scan_map<T, VEC>(dy + ((long long)(n0 + (live ? i : 0)) * g.k + k) * pq, live, pq, G, sub, best_j, s);
            if (live && sub == 0) put_record(i, i, best_j, s);
        }
    }
    const int nrec = cnt * topk;           // records of this CTA: one per image, or topk per image
    __syncthreads();

    // ---- phase 2: patch accumulate ----
    // A work item is (element group, image lane j): NJ lanes (chosen by the host: enough that a lane has at
    // most eight images and that no thread idles) split the images round-robin
    // (i = j, j+NJ, ...), each adding its images in ascending order with up to eight loads in flight;
    // the NJ subtotals are then added in lane order.  VX elements per group: four channels per load
    // on the vector path (NHWC, C a multiple of four), else one.
    {
        // WIDE (bf16, C a multiple of eight): eight channels per 16-byte load, four loads in flight
        const int VX = WIDE ? 8 : vec_x ? 4 : 1;
        constexpr int BATCH = (sizeof(T) == 4 || WIDE) ? 4 : 8;          // loads in flight per thread (register budget: 64)
        constexpr int NV = WIDE ? 8 : 4;
        const int groups = rsc / VX;
        float* s_sub = NJ > 1 ? s_subs : s_part;               // NJ == 1: results go straight to s_part
        for (int item = threadIdx.x; item < groups * NJ; item += blockDim.x) {
            const int j = item / groups, e = (item - j * groups) * VX;
            const int c = e % g.c, rs = e / g.c, s = rs % g.s, r = rs / g.s;
            const T* xc = x + n0 * g.xs_n + c * g.xs_c + r * g.xs_h + s * g.xs_w;     // this element of a patch whose corner is pixel (0,0)
            const uint32_t bits = (1u << r) | (1u << (16 + s));
            float acc[NV];
#pragma unroll
            for (int t = 0; t < NV; ++t) acc[t] = 0.f;
            for (int i0 = j; i0 < nrec; i0 += BATCH * NJ) {
                // BATCH loads are issued before any is consumed; they stay raw (two or four registers each)
                // until then, so that the register allocator has no reason to serialise them.  A patch element
                // outside the image contributes weight 0 times a zero that is not loaded.
                Raw4 raw[BATCH];
                float wsum[BATCH];
#pragma unroll
                for (int u = 0; u < BATCH; ++u) {
                    const int i = i0 + u * NJ;
                    const bool in = i < nrec;
                    const uint4 rec = s_rec[in ? i : 0];
                    const bool ok = in && (rec.w & bits) == bits;
                    wsum[u] = ok ? __uint_as_float(rec.z) : 0.f;
                    const T* p = xc + (long long)(((unsigned long long)rec.y << 32) | rec.x);
                    raw[u] = Raw4{{0u, 0u, 0u, 0u}};
                    if (ok) {
                        if (WIDE) raw[u] = ld8_raw(p);
                        else if (vec_x) raw[u] = ld4_raw(p);
                        else raw[u].w[0] = __float_as_uint(ldf(p));
                    }
                }
#pragma unroll
                for (int u = 0; u < BATCH; ++u) {
                    float v[NV];
                    if constexpr (WIDE) raw_to_float8(raw[u], v);
                    else {
                        float v4[4];
                        if (vec_x) raw_to_float(raw[u], static_cast<const T*>(nullptr), v4);
                        else { v4[0] = __uint_as_float(raw[u].w[0]); v4[1] = v4[2] = v4[3] = 0.f; }
#pragma unroll
                        for (int t = 0; t < 4; ++t) v[t] = v4[t];
                    }
#pragma unroll
                    for (int t = 0; t < NV; ++t) acc[t] = fmaf(wsum[u], v[t], acc[t]);
                }
            }
            float* out = s_sub + j * rsc + e;
            if (VX >= 4) {            // 16-byte stores: rsc and e are multiples of four here
                *reinterpret_cast<float4*>(out) = make_float4(acc[0], acc[1], acc[2], acc[3]);
                if constexpr (WIDE) *reinterpret_cast<float4*>(out + 4) = make_float4(acc[4], acc[5], acc[6], acc[7]);
            } else {
                out[0] = acc[0];
            }
        }
        if (NJ > 1) {
            __syncthreads();
            for (int e = threadIdx.x; e < rsc; e += blockDim.x) {
                float tot = s_sub[e];
                for (int j = 1; j < NJ; ++j) tot += s_sub[j * rsc + e];
                s_part[e] = tot;
            }
        }
    }
    cluster.sync();

    // ---- phase 3: rank j finishes slice j ----
    const int slice = (rsc + CL - 1) / CL;
    const int e_end = min(rsc, (chunk + 1) * slice);
    for (int e = chunk * slice + threadIdx.x; e < e_end; e += blockDim.x) {
        float pv[8];
#pragma unroll
        for (int rk = 0; rk < 8; ++rk) pv[rk] = rk < CL ? *cluster.map_shared_rank(s_part + e, rk) : 0.0f;
        float tot = 0.0f;
#pragma unroll
        for (int rk = 0; rk < 8; ++rk) tot += pv[rk];          // rank order; absent ranks add +0
        const int c = e % g.c, rs = e / g.c, s = rs % g.s, r = rs / g.s;
        dw[k * g.ws_k + c * g.ws_c + r * g.ws_r + s * g.ws_s] = g.alpha * tot;
    }
    cluster.sync();     // peers may still be reading this CTA's block
#ifdef GACONV_TUNING
    if (logger) gaconv_tuning_top1_log[log_i][2] = tuning_now();
#endif
}

// grid (chunks, K).  Each CTA owns the images [chunk*ipc, (chunk+1)*ipc) of one output channel and
// accumulates their patches in image order (topk retained entries per map, each weighted sum/topk; topk = 1
// is Algorithm 1); the last CTA of a channel to finish adds the per-chunk partials in chunk order (fixed
// order => reproducible) and writes dW.
template <typename T>
__global__ void __launch_bounds__(256)
gather_kernel(const T* __restrict__ x, const int32_t* __restrict__ idx, const float* __restrict__ sum,
              float* __restrict__ dw, float* __restrict__ partial, uint32_t* __restrict__ counters, Geom g,
              int chunks, int ipc, int topk)
{
    pdl_release_next_grid();
    pdl_wait_prior_grid();
    extern __shared__ int smem_i[];
    int* s_h0 = smem_i;                       // top-left input row of each retained entry's patch, [image][topk]
    int* s_w0 = smem_i + ipc * topk;
    float* s_sum = reinterpret_cast<float*>(smem_i + 2 * ipc * topk);   // [image]: sum / topk
    __shared__ bool s_last;

    const int k = blockIdx.y, chunk = blockIdx.x;
    const int n0 = chunk * ipc;
    const int cnt = min(ipc, g.n - n0);
    for (int it = threadIdx.x; it < cnt * topk; it += blockDim.x) {
        const int i = it / topk;
        const long long m = (long long)(n0 + i) * g.k + k;
        const int j = idx[m * topk + (it - i * topk)];
        s_h0[it] = (j / g.q) * g.stride_h - g.pad_h;
        s_w0[it] = (j % g.q) * g.stride_w - g.pad_w;
        if (it == i * topk) s_sum[i] = sum[m] / (float)topk;
    }
    __syncthreads();

    const int rsc = g.r * g.s * g.c;
    float* part = partial + ((size_t)chunk * g.k + k) * rsc;
    for (int e = threadIdx.x; e < rsc; e += blockDim.x) {
        const int c = e % g.c, rs = e / g.c, s = rs % g.s, r = rs / g.s;
        float acc = 0.0f;
        for (int i = 0; i < cnt; ++i)
            for (int t = 0; t < topk; ++t) {
                const int hh = s_h0[i * topk + t] + r, ww = s_w0[i * topk + t] + s;
                if (hh >= 0 && hh < g.h && ww >= 0 && ww < g.w)
                    acc = fmaf(s_sum[i], ldf(x + (n0 + i) * g.xs_n + c * g.xs_c + hh * g.xs_h + ww * g.xs_w), acc);
            }
        if (chunks == 1) dw[k * g.ws_k + c * g.ws_c + r * g.ws_r + s * g.ws_s] = g.alpha * acc;
        else part[e] = acc;
    }
    if (chunks == 1) return;

    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t ticket = atomicAdd(&counters[k % kWsNumCounters], 1u);
        s_last = (ticket == (uint32_t)chunks - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    for (int e = threadIdx.x; e < rsc; e += blockDim.x) {
        const int c = e % g.c, rs = e / g.c, s = rs % g.s, r = rs / g.s;
        float tot = 0.0f;
        for (int ch = 0; ch < chunks; ++ch) tot += __ldcg(partial + ((size_t)ch * g.k + k) * rsc + e);
        dw[k * g.ws_k + c * g.ws_c + r * g.ws_r + s * g.ws_s] = g.alpha * tot;
    }
    if (threadIdx.x == 0) counters[k % kWsNumCounters] = 0;   // leave the counters as found
}

int pow2_floor(int v) { int p = 1; while (p * 2 <= v) p *= 2; return p; }

struct MapScanShape { bool vec; int G; };
MapScanShape map_scan_shape(const Geom& g)
{
    const int pq = g.p * g.q, eb = g.bf16 ? 2 : 4;
    MapScanShape m;
    m.vec = ((size_t)pq * eb) % 16 == 0;
    const int units = m.vec ? pq * eb / 16 : pq;
    m.G = pow2_floor(units);
    if (m.G > 32) m.G = 32;
    return m;
}

}  // namespace

cudaError_t launch_select(const void* dy, int32_t* idx, float* sum, void* dy_sparse, const Geom& g,
                          cudaStream_t stream)
{
    const long long maps = (long long)g.n * g.k;
    const int pq = g.p * g.q;
    const MapScanShape m = map_scan_shape(g);
    const int maps_per_cta = (256 / 32) * (32 / m.G);
    const unsigned grid = (unsigned)((maps + maps_per_cta - 1) / maps_per_cta);
    if (g.bf16) {
        auto d = static_cast<const __nv_bfloat16*>(dy); auto o = static_cast<__nv_bfloat16*>(dy_sparse);
        if (m.vec) select_kernel<__nv_bfloat16, true><<<grid, 256, 0, stream>>>(d, idx, sum, o, maps, pq, m.G);
        else       select_kernel<__nv_bfloat16, false><<<grid, 256, 0, stream>>>(d, idx, sum, o, maps, pq, m.G);
    } else {
        auto d = static_cast<const float*>(dy); auto o = static_cast<float*>(dy_sparse);
        if (m.vec) select_kernel<float, true><<<grid, 256, 0, stream>>>(d, idx, sum, o, maps, pq, m.G);
        else       select_kernel<float, false><<<grid, 256, 0, stream>>>(d, idx, sum, o, maps, pq, m.G);
    }
    note_launch();
    return cudaGetLastError();
}

cudaError_t launch_select_sparse_transposed(const void* dy, void* dyt, const Geom& g, cudaStream_t stream)
{
    cudaError_t e = launch_kernel(select_sparse_transposed_kernel, dim3((unsigned)(g.n * ((g.k + 63) / 64))), dim3(128), 0, stream, dim3(1, 1, 1),
                                  static_cast<const __nv_bfloat16*>(dy), static_cast<__nv_bfloat16*>(dyt), g.k, g.p * g.q);
    note_launch();
    return e;
}

cudaError_t launch_select_topk(const void* dy, int32_t* idx, float* sum, const Geom& g, int topk, cudaStream_t stream)
{
    const long long maps = (long long)g.n * g.k;
    const unsigned grid = (unsigned)((maps + 7) / 8);
    if (g.bf16) select_topk_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(dy), idx, sum, maps, g.p * g.q, topk);
    else        select_topk_kernel<float><<<grid, 256, 0, stream>>>(static_cast<const float*>(dy), idx, sum, maps, g.p * g.q, topk);
    note_launch();
    return cudaGetLastError();
}

GatherPlan plan_gather(const Geom& g)
{
    GatherPlan p;
    // enough CTAs to cover the SMs a few times over, while keeping the partial buffer small
    const size_t out_bytes = (size_t)g.k * g.r * g.s * g.c * sizeof(float);
    int chunks = (4 * 148 + g.k - 1) / g.k;
    if (chunks > g.n) chunks = g.n;
    while (chunks > 1 && chunks * out_bytes > ((size_t)32 << 20)) --chunks;
    if (chunks < 1) chunks = 1;
    p.imgs_per_chunk = (g.n + chunks - 1) / chunks;
    p.chunks = (g.n + p.imgs_per_chunk - 1) / p.imgs_per_chunk;
    p.partial_bytes = p.chunks > 1 ? p.chunks * out_bytes : 0;
    return p;
}

cudaError_t launch_gather(const void* x, const int32_t* idx, const float* sum, float* dw, float* partial,
                          uint32_t* counters, const Geom& g, const GatherPlan& plan, int topk, cudaStream_t stream)
{
    dim3 grid(plan.chunks, g.k);
    const size_t smem = (size_t)plan.imgs_per_chunk * (8 * topk + 4);
    if (smem > 48 * 1024) return cudaErrorInvalidValue;
    if (g.bf16)
        gather_kernel<__nv_bfloat16><<<grid, 256, smem, stream>>>(static_cast<const __nv_bfloat16*>(x), idx, sum, dw,
                                                                   partial, counters, g, plan.chunks, plan.imgs_per_chunk, topk);
    else
        gather_kernel<float><<<grid, 256, smem, stream>>>(static_cast<const float*>(x), idx, sum, dw, partial,
                                                          counters, g, plan.chunks, plan.imgs_per_chunk, topk);
    note_launch();
    return cudaGetLastError();
}

bool top1_fused_supported(const Geom& g)
{
    // the per-channel block of R*S*C sums lives in shared memory
    return (size_t)g.r * g.s * g.c * sizeof(float) <= 100 * 1024 && g.k <= 65535 && g.r <= 16 && g.s <= 16;
}

template <typename T, bool VEC, bool WIDE>
static cudaError_t launch_fused_t(const T* x, const T* dy, float* dw, const Geom& g, int cl, int ipc, int G, cudaStream_t stream,
                                  const int32_t* sel_idx = nullptr, const float* sel_sum = nullptr, int topk = 1)
{
    // block of sums + per-image arrays + up to 16 lane subtotals when the block is small
    const int rsc = g.r * g.s * g.c;
    const bool vec_x = g.xs_c == 1 && g.c % 4 == 0;
    int nj = 1;
    // 512 threads (two CTAs per SM) where the grid still fits in one wave and the scan would otherwise need
    // two passes over the CTA's maps; measured: helps 32-channel layers, neutral or worse for 16 and 64
    const int threads = (g.sm_budget == 0 && g.k >= 32 && (long long)cl * g.k <= 148 * 2) ? 512 : 256;
    const int groups = rsc / (WIDE ? 8 : vec_x ? 4 : 1);
    const int batch = (sizeof(T) == 4 || WIDE) ? 4 : 8;
    (void)batch;
    while (nj < 16 && nj * 2 <= ipc * topk && nj * 2 * groups <= threads) nj *= 2;        // image lanes: as many as keep every item on its own thread
    while (nj > 1 && (size_t)rsc * 4 * (1 + nj) > 150 * 1024) nj /= 2;              // the subtotals must fit shared memory
    const size_t smem = (((size_t)rsc * 4 + 15) & ~(size_t)15) + (size_t)ipc * topk * 16 + (nj > 1 ? (size_t)nj * rsc * 4 : 0) + 16;
    static size_t configured[64] = {};           // per device: the attribute belongs to the device's copy of the kernel
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (smem > 48 * 1024 && smem > configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(top1_fused_kernel<T, VEC, WIDE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured[dev] = smem;
    }
    // lanes per map: few enough that one pass covers all the CTA's maps (their loads are then all in flight at once)
    while (G > 1 && G * ipc > threads) G /= 2;
    cudaError_t e = launch_kernel(top1_fused_kernel<T, VEC, WIDE>, dim3(cl, g.k), dim3(threads), smem, stream, dim3(cl, 1, 1), x, dy, dw, g, ipc, G, vec_x, nj,
                                  sel_idx, sel_sum, topk);
    note_launch();
    return e;
}

#ifdef GACONV_TUNING
}  // namespace gaconv
extern "C" int gaconv_tuning_read_top1_log(unsigned long long* host, unsigned int* count)
{
    if (cudaMemcpyFromSymbol(count, gaconv::gaconv_tuning_top1_log_n, sizeof(unsigned int)) != cudaSuccess) return 1;
    return (int)cudaMemcpyFromSymbol(host, gaconv::gaconv_tuning_top1_log, sizeof(gaconv::gaconv_tuning_top1_log));
}
namespace gaconv {
#endif

// sel_idx != nullptr: the top-k method -- selection was done by launch_select_topk; the kernel accumulates topk records per image
cudaError_t launch_top1_fused(const void* x, const void* dy, float* dw, const Geom& g, cudaStream_t stream,
                              const int32_t* sel_idx, const float* sel_sum, int topk)
{
    int cl = 1;
    while (cl * 2 <= 8 && cl * 2 <= g.n) cl *= 2;
    // fewer, fatter CTAs when there are already plenty of channels: the whole grid should be resident
    // at once (four CTAs of 64 registers x 256 threads fit an SM)
    while (cl > 1 && (long long)cl * g.k > 148 * 4) cl /= 2;
    // sharing the GPU with other layers (the caller gave an SM budget): about four CTAs per budgeted SM, so that the
    // registers of several such kernels fit next to one another
    if (g.sm_budget > 0)
        while (cl > 1 && (long long)cl * g.k > 4LL * g.sm_budget) cl /= 2;
    const int ipc = (g.n + cl - 1) / cl;
    const MapScanShape m = map_scan_shape(g);
    if (g.bf16) {
        auto xx = static_cast<const __nv_bfloat16*>(x); auto dd = static_cast<const __nv_bfloat16*>(dy);
        const bool wide = g.xs_c == 1 && g.c % 8 == 0 && g.xs_w % 8 == 0;     // 16-byte aligned groups of eight channels
        if (wide) return m.vec ? launch_fused_t<__nv_bfloat16, true, true>(xx, dd, dw, g, cl, ipc, m.G, stream, sel_idx, sel_sum, topk)
                               : launch_fused_t<__nv_bfloat16, false, true>(xx, dd, dw, g, cl, ipc, m.G, stream, sel_idx, sel_sum, topk);
        return m.vec ? launch_fused_t<__nv_bfloat16, true, false>(xx, dd, dw, g, cl, ipc, m.G, stream, sel_idx, sel_sum, topk)
                     : launch_fused_t<__nv_bfloat16, false, false>(xx, dd, dw, g, cl, ipc, m.G, stream, sel_idx, sel_sum, topk);
    }
    auto xx = static_cast<const float*>(x); auto dd = static_cast<const float*>(dy);
    return m.vec ? launch_fused_t<float, true, false>(xx, dd, dw, g, cl, ipc, m.G, stream, sel_idx, sel_sum, topk)
                 : launch_fused_t<float, false, false>(xx, dd, dw, g, cl, ipc, m.G, stream, sel_idx, sel_sum, topk);
}

}  // namespace gaconv
