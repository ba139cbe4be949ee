// Max-gradient approximation (paper Section 2.3, Algorithm 1) as two kernels:
//   select_kernel  -- per (n,k) map of dY: position of the largest magnitude (lowest index among
//                     equals) and the signed sum of the map      [Algorithm 1, arg-max and sum lines]
//   gather_kernel  -- dW[k,r,s,c] = alpha * sum_n sum[n,k] * Xz[n, c, patch at the selected position]
//                                                                  [Algorithm 1, accumulation line]
// Selection compares the bit pattern of |v| in the input dtype as an unsigned integer, which orders
// finite values exactly as their magnitudes do, so indices are reproducible bit for bit.
#include "gaconv_internal.h"

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

// One group of G lanes (G a power of two, G <= 32) scans one map.  VEC: 16-byte loads (maps are a
// whole number of 16-byte vectors and therefore 16-byte aligned) or element loads.
template <typename T, bool VEC>
__global__ void __launch_bounds__(256)
select_kernel(const T* __restrict__ dy, int32_t* __restrict__ idx, float* __restrict__ sum,
              T* __restrict__ dy_sparse, long long num_maps, int pq, int G)
{
    const int lane = threadIdx.x & 31;
    const int sub = lane & (G - 1);
    const int maps_per_warp = 32 / G;
    const long long warp = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long long m = warp * maps_per_warp + lane / G;
    const bool live = m < num_maps;
    Scan sc{-1, 0, 0.0f};
    const T* map = dy + (live ? m : 0) * (long long)pq;
    if (live) {
        if (VEC) {
            constexpr int E = Elem<T>::kPerVec;
            const uint4* mv = reinterpret_cast<const uint4*>(map);
            const int nvec = pq / E;
            int v = sub;
            // four independent loads in flight per lane before any is consumed
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
    // combine the G lanes: larger magnitude wins, then the lower index; sums add in a fixed tree
    unsigned long long key = ((unsigned long long)(unsigned)(sc.best_mag + 1) << 32) | (0xffffffffu - (unsigned)sc.best_j);
    float s = sc.sum;
    for (int off = G >> 1; off > 0; off >>= 1) {
        unsigned long long other = __shfl_xor_sync(0xffffffffu, key, off);
        float so = __shfl_xor_sync(0xffffffffu, s, off);
        key = other > key ? other : key;
        s += so;
    }
    if (!live) return;
    const int best_j = (int)(0xffffffffu - (unsigned)(key & 0xffffffffu));
    if (sub == 0) { idx[m] = best_j; sum[m] = s; }
    if (dy_sparse != nullptr) {
        T* out = dy_sparse + m * (long long)pq;
        for (int j = sub; j < pq; j += G) Elem<T>::store1(out + j, j == best_j ? s : 0.0f);
    }
}

template <typename T> __device__ __forceinline__ float ld_as_float(const T* p);
template <> __device__ __forceinline__ float ld_as_float<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float ld_as_float<__nv_bfloat16>(const __nv_bfloat16* p) {
    return bf16_bits_to_float(__ldg(reinterpret_cast<const unsigned short*>(p)));
}

// grid (chunks, K).  Each CTA owns the images [chunk*ipc, (chunk+1)*ipc) of one output channel and
// accumulates their patches in image order; the last CTA of a channel to finish adds the per-chunk
// partials in chunk order (fixed order => reproducible) and writes dW.
template <typename T>
__global__ void __launch_bounds__(256)
gather_kernel(const T* __restrict__ x, const int32_t* __restrict__ idx, const float* __restrict__ sum,
              float* __restrict__ dw, float* __restrict__ partial, uint32_t* __restrict__ counters, Geom g,
              int chunks, int ipc)
{
    extern __shared__ int smem_i[];
    int* s_h0 = smem_i;                       // top-left input row of each image's patch
    int* s_w0 = smem_i + ipc;
    float* s_sum = reinterpret_cast<float*>(smem_i + 2 * ipc);
    __shared__ bool s_last;

    const int k = blockIdx.y, chunk = blockIdx.x;
    const int n0 = chunk * ipc;
    const int cnt = min(ipc, g.n - n0);
    for (int i = threadIdx.x; i < cnt; i += blockDim.x) {
        const long long m = (long long)(n0 + i) * g.k + k;
        const int j = idx[m];
        s_h0[i] = (j / g.q) * g.stride_h - g.pad_h;
        s_w0[i] = (j % g.q) * g.stride_w - g.pad_w;
        s_sum[i] = sum[m];
    }
    __syncthreads();

    const int rsc = g.r * g.s * g.c;
    float* part = partial + ((size_t)chunk * g.k + k) * rsc;
    for (int e = threadIdx.x; e < rsc; e += blockDim.x) {
        const int c = e % g.c, rs = e / g.c, s = rs % g.s, r = rs / g.s;
        float acc = 0.0f;
        for (int i = 0; i < cnt; ++i) {
            const int hh = s_h0[i] + r, ww = s_w0[i] + s;
            if (hh >= 0 && hh < g.h && ww >= 0 && ww < g.w)
                acc = fmaf(s_sum[i], ld_as_float(x + (n0 + i) * g.xs_n + c * g.xs_c + hh * g.xs_h + ww * g.xs_w), acc);
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

}  // namespace

cudaError_t launch_select(const void* dy, int32_t* idx, float* sum, void* dy_sparse, const Geom& g,
                          cudaStream_t stream)
{
    const long long maps = (long long)g.n * g.k;
    const int pq = g.p * g.q;
    const int eb = g.bf16 ? 2 : 4;
    const bool vec = ((size_t)pq * eb) % 16 == 0;
    const int units = vec ? pq * eb / 16 : pq;
    int G = pow2_floor(units); if (G > 32) G = 32;
    const int maps_per_cta = (256 / 32) * (32 / G);
    const unsigned grid = (unsigned)((maps + maps_per_cta - 1) / maps_per_cta);
    if (g.bf16) {
        auto d = static_cast<const __nv_bfloat16*>(dy); auto o = static_cast<__nv_bfloat16*>(dy_sparse);
        if (vec) select_kernel<__nv_bfloat16, true><<<grid, 256, 0, stream>>>(d, idx, sum, o, maps, pq, G);
        else     select_kernel<__nv_bfloat16, false><<<grid, 256, 0, stream>>>(d, idx, sum, o, maps, pq, G);
    } else {
        auto d = static_cast<const float*>(dy); auto o = static_cast<float*>(dy_sparse);
        if (vec) select_kernel<float, true><<<grid, 256, 0, stream>>>(d, idx, sum, o, maps, pq, G);
        else     select_kernel<float, false><<<grid, 256, 0, stream>>>(d, idx, sum, o, maps, pq, G);
    }
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
                          uint32_t* counters, const Geom& g, const GatherPlan& plan, cudaStream_t stream)
{
    dim3 grid(plan.chunks, g.k);
    const size_t smem = (size_t)plan.imgs_per_chunk * 12;
    if (g.bf16)
        gather_kernel<__nv_bfloat16><<<grid, 256, smem, stream>>>(static_cast<const __nv_bfloat16*>(x), idx, sum, dw,
                                                                   partial, counters, g, plan.chunks, plan.imgs_per_chunk);
    else
        gather_kernel<float><<<grid, 256, smem, stream>>>(static_cast<const float*>(x), idx, sum, dw, partial,
                                                          counters, g, plan.chunks, plan.imgs_per_chunk);
    note_launch();
    return cudaGetLastError();
}

}  // namespace gaconv
