// Global-memory access helpers and launch sizing shared by the streaming kernels (one pass over
// the data, every byte touched once).
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace adama {

// ---- 128-bit global accesses ------------------------------------------------------------
// m, v and w are read once and written once per pass, the gradient is read once:
// loads do not allocate in L1.
__device__ __forceinline__ float4 ld_stream(const float4 *p) {
    float4 r;
    asm volatile("ld.global.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w)
                 : "l"(p));
    return r;
}
__device__ __forceinline__ uint2 ld_stream_ro(const uint2 *p) {
    uint2 r;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(r.x), "=r"(r.y) : "l"(p));
    return r;
}
__device__ __forceinline__ float4 ld_stream_ro(const float4 *p) {
    float4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w)
                 : "l"(p));
    return r;
}
__device__ __forceinline__ void st_stream(float4 *p, float4 x) {
#ifdef ADAMA_ST_CS
    asm volatile("st.global.cs.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(p), "f"(x.x), "f"(x.y), "f"(x.z),
                 "f"(x.w)
                 : "memory");
    return;
#endif
    asm volatile("st.global.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(p), "f"(x.x), "f"(x.y), "f"(x.z),
                 "f"(x.w)
                 : "memory");
}

// four gradient values widened exactly to fp32
struct Grad4 {
    float x, y, z, w;
};
__device__ __forceinline__ Grad4 load_grad4(const float *g, size_t i4) {
    float4 t = ld_stream_ro(reinterpret_cast<const float4 *>(g) + i4);
    return {t.x, t.y, t.z, t.w};
}
__device__ __forceinline__ Grad4 load_grad4(const __nv_bfloat16 *g, size_t i4) {
    uint2 t = ld_stream_ro(reinterpret_cast<const uint2 *>(g) + i4);
    // bf16 -> fp32 is a 16-bit left shift
    return {__uint_as_float(t.x << 16), __uint_as_float(t.x & 0xffff0000u),
            __uint_as_float(t.y << 16), __uint_as_float(t.y & 0xffff0000u)};
}
__device__ __forceinline__ float widen(float g) { return g; }
__device__ __forceinline__ float widen(__nv_bfloat16 g) { return __bfloat162float(g); }

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Grid: enough CTAs to cover the data once, capped at a whole number of CTAs per SM.
inline unsigned grid_for(size_t work_items, size_t items_per_cta, int sm_count, int ctas_per_sm) {
    size_t need = (work_items + items_per_cta - 1) / items_per_cta;
    size_t cap = (size_t)sm_count * ctas_per_sm;
    if (need < 1) need = 1;
    return (unsigned)(need < cap ? need : cap);
}

}  // namespace adama
