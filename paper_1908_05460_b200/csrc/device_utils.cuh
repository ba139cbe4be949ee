// Small device helpers shared by the kernels: element loads with conversion to fp32, the TF32 split, and
// the warp-level MMA instructions.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace gaconv {

// one element as fp32
__device__ __forceinline__ float ldf(const float* p) { return __ldg(p); }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p) {
    return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p)) << 16);
}

// four consecutive elements as fp32 (16-byte load for fp32, 8-byte load for bf16; p aligned accordingly)
__device__ __forceinline__ void ld4(const float* p, float (&v)[4]) {
    const float4 t = __ldg(reinterpret_cast<const float4*>(p));
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
__device__ __forceinline__ void ld4(const __nv_bfloat16* p, float (&v)[4]) {
    const uint2 t = __ldg(reinterpret_cast<const uint2*>(p));
    v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xffff0000u);
    v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xffff0000u);
}

// TF32 value of v by truncation (low 13 mantissa bits cleared): one full-rate logic op instead of a trip
// through the conversion unit.  The split x = big + small (big = to_tf32(x), small = to_tf32(x - big)) stays
// exact up to 2^-20 |x|, and big*big + big*small + small*big reproduces an fp32 product to ~2^-21.
__device__ __forceinline__ uint32_t to_tf32(float v) { return __float_as_uint(v) & 0xffffe000u; }

// D += A*B on the warp-level tensor-core path; fragment layouts as in the PTX ISA (row.col)
__device__ __forceinline__ void mma_tf32(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

}  // namespace gaconv
