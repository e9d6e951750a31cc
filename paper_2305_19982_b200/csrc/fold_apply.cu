// Streaming kernels of AdamA: the moment fold (Algorithm 2, inner loop body) and
// the update fused with the next mini-batch's decay (Algorithm 2, "Update" and the
// first line of the loop body).  Both are pure HBM streams: one pass, every byte
// touched once, 128-bit coalesced accesses, several independent loads in flight
// per thread, grid sized as a multiple of the SM count with a grid-stride loop.
#include <cuda_bf16.h>

#include "adama_device.cuh"
#include "stream_access.cuh"

namespace adama {
namespace {

// Launch shape.  Measured on B200 at 335 M
// parameters: one fat CTA per SM with many independent 128-bit loads per thread beats
// several thin ones -- fold 6.28 TB/s at (256 threads, unroll 6, 1 CTA/SM) against 6.03 at
// (unroll 4, 4 CTAs/SM); apply 6.30 TB/s at (8 groups, 1 CTA/SM) against 5.81 at (4, 3).
constexpr int kThreads = 256;
constexpr int kFoldUnroll = 6;      // fold: 6 x (g, m, v) vectors in flight per thread
constexpr int kApplyUnroll = 4;     // apply: 2 x 4 x (w, m, v) vectors = 96 data registers
constexpr int kCtasPerSm = 1;
constexpr int kApplyCtasPerSm = 1;

template <typename G, int UNROLL>
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
fold_vec_kernel(const G *__restrict__ grad, float *__restrict__ m, float *__restrict__ v,
                size_t n4, size_t n, float a, float b) {
    float4 *m4 = reinterpret_cast<float4 *>(m);
    float4 *v4 = reinterpret_cast<float4 *>(v);
    const size_t span = (size_t)kThreads * UNROLL;
    for (size_t base = (size_t)blockIdx.x * span; base < n4; base += (size_t)gridDim.x * span) {
        Grad4 g[UNROLL];
        float4 mm[UNROLL], vv[UNROLL];
        // all loads of the iteration are issued before the first use
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            size_t i = base + (size_t)u * kThreads + threadIdx.x;
            if (i < n4) {
                g[u] = load_grad4(grad, i);
                mm[u] = ld_stream(m4 + i);
                vv[u] = ld_stream(v4 + i);
            }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            size_t i = base + (size_t)u * kThreads + threadIdx.x;
            if (i < n4) {
                fold1(g[u].x, mm[u].x, vv[u].x, a, b);
                fold1(g[u].y, mm[u].y, vv[u].y, a, b);
                fold1(g[u].z, mm[u].z, vv[u].z, a, b);
                fold1(g[u].w, mm[u].w, vv[u].w, a, b);
                st_stream(m4 + i, mm[u]);
                st_stream(v4 + i, vv[u]);
            }
        }
    }
    // ragged tail (n not a multiple of 4): at most 3 elements
    if (blockIdx.x == 0 && threadIdx.x < (unsigned)(n - n4 * 4)) {
        size_t i = n4 * 4 + threadIdx.x;
        float mi = m[i], vi = v[i];
        fold1(widen(grad[i]), mi, vi, a, b);
        m[i] = mi;
        v[i] = vi;
    }
}

// Fallback for pointers that are not 16-byte aligned (8-byte for bf16 gradients).
template <typename G>
__global__ void __launch_bounds__(kThreads)
fold_scalar_kernel(const G *__restrict__ grad, float *__restrict__ m, float *__restrict__ v,
                   size_t n, float a, float b) {
    for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < n;
         i += (size_t)gridDim.x * kThreads) {
        float mi = m[i], vi = v[i];
        fold1(widen(grad[i]), mi, vi, a, b);
        m[i] = mi;
        v[i] = vi;
    }
}

// two fp32 -> packed bf16x2, round to nearest even
__device__ __forceinline__ unsigned pack_bf16x2(float lo, float hi) {
    const __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const unsigned *>(&p);
}

// COPY: also write the updated weights rounded to bf16 (the copy a mixed-precision forward
// pass reads), 2 B/param on top of the 24, instead of a separate cast pass of 6 B/param.
//
// Software-pipelined: two register buffers of UNROLL {w, m, v} vector groups; the loads of the
// NEXT span are issued before the arithmetic and the stores of the current one, so reads and
// writes reach the memory system interleaved instead of in alternating bursts.  Measured at
// 335 M parameters: 1.286 ms (2 x 4 groups) against 1.33-1.34 ms for one buffer of 8 groups
// with all loads first; 2 x 3: 1.42, 2 x 5: 1.30, 2 x 6: 1.33 ms.  (The fold did not gain
// from the same change: 2 x 3 groups 1.12 ms, 2 x 4 1.02 ms against 0.96 ms for 1 x 6.)
template <int UNROLL, bool COPY>
__global__ void __launch_bounds__(kThreads, kApplyCtasPerSm)
apply_vec_kernel(float *__restrict__ w, float *__restrict__ m, float *__restrict__ v,
                 __nv_bfloat16 *__restrict__ w_bf16, size_t n4, size_t n, ApplyConstants c) {
    float4 *w4 = reinterpret_cast<float4 *>(w);
    float4 *m4 = reinterpret_cast<float4 *>(m);
    float4 *v4 = reinterpret_cast<float4 *>(v);
    const size_t span = (size_t)kThreads * UNROLL;
    const size_t stride = (size_t)gridDim.x * span;
    float4 ww[2][UNROLL], mm[2][UNROLL], vv[2][UNROLL];
    size_t base = (size_t)blockIdx.x * span;
    if (base < n4) {
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            size_t i = base + (size_t)u * kThreads + threadIdx.x;
            if (i < n4) {
                ww[0][u] = ld_stream(w4 + i);
                mm[0][u] = ld_stream(m4 + i);
                vv[0][u] = ld_stream(v4 + i);
            }
        }
    }
#pragma unroll 1
    for (; base < n4; base += 2 * stride) {
#pragma unroll
        for (int buf = 0; buf < 2; ++buf) {
            const size_t cur = base + (size_t)buf * stride;
            const size_t nxt = cur + stride;
            if (cur < n4) {
                if (nxt < n4) {
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) {
                        size_t i = nxt + (size_t)u * kThreads + threadIdx.x;
                        if (i < n4) {
                            ww[buf ^ 1][u] = ld_stream(w4 + i);
                            mm[buf ^ 1][u] = ld_stream(m4 + i);
                            vv[buf ^ 1][u] = ld_stream(v4 + i);
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    size_t i = cur + (size_t)u * kThreads + threadIdx.x;
                    if (i < n4) {
                        float4 &x = ww[buf][u], &y = mm[buf][u], &z = vv[buf][u];
                        apply1(x.x, y.x, z.x, c);
                        apply1(x.y, y.y, z.y, c);
                        apply1(x.z, y.z, z.z, c);
                        apply1(x.w, y.w, z.w, c);
                        st_stream(w4 + i, x);
                        st_stream(m4 + i, y);
                        st_stream(v4 + i, z);
                        if (COPY)
                            reinterpret_cast<uint2 *>(w_bf16)[i] =
                                make_uint2(pack_bf16x2(x.x, x.y), pack_bf16x2(x.z, x.w));
                    }
                }
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x < (unsigned)(n - n4 * 4)) {
        size_t i = n4 * 4 + threadIdx.x;
        float wi = w[i], mi = m[i], vi = v[i];
        apply1(wi, mi, vi, c);
        w[i] = wi;
        m[i] = mi;
        v[i] = vi;
        if (COPY) w_bf16[i] = __float2bfloat16_rn(wi);
    }
}

__global__ void __launch_bounds__(kThreads)
apply_scalar_kernel(float *__restrict__ w, float *__restrict__ m, float *__restrict__ v,
                    __nv_bfloat16 *__restrict__ w_bf16, size_t n, ApplyConstants c) {
    for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < n;
         i += (size_t)gridDim.x * kThreads) {
        float wi = w[i], mi = m[i], vi = v[i];
        apply1(wi, mi, vi, c);
        w[i] = wi;
        m[i] = mi;
        v[i] = vi;
        if (w_bf16) w_bf16[i] = __float2bfloat16_rn(wi);
    }
}

}  // namespace

cudaError_t launch_fold(const void *grad, adama_dtype gdt, float *m, float *v, size_t n,
                        FoldConstants c, int sm_count, cudaStream_t stream) {
    if (n == 0) return cudaSuccess;
    constexpr int U = kFoldUnroll;
    const size_t n4 = n / 4;
    const bool vec = aligned(m, 16) && aligned(v, 16) && aligned(grad, gdt == ADAMA_F32 ? 16 : 8);
    if (gdt == ADAMA_F32) {
        const float *g = static_cast<const float *>(grad);
        if (vec) {
            unsigned grid = grid_for(n4, (size_t)kThreads * U, sm_count, kCtasPerSm);
            fold_vec_kernel<float, U><<<grid, kThreads, 0, stream>>>(g, m, v, n4, n, c.a, c.b);
        } else {
            unsigned grid = grid_for(n, kThreads, sm_count, kCtasPerSm);
            fold_scalar_kernel<float><<<grid, kThreads, 0, stream>>>(g, m, v, n, c.a, c.b);
        }
    } else {
        const __nv_bfloat16 *g = static_cast<const __nv_bfloat16 *>(grad);
        if (vec) {
            unsigned grid = grid_for(n4, (size_t)kThreads * U, sm_count, kCtasPerSm);
            fold_vec_kernel<__nv_bfloat16, U><<<grid, kThreads, 0, stream>>>(g, m, v, n4, n, c.a,
                                                                              c.b);
        } else {
            unsigned grid = grid_for(n, kThreads, sm_count, kCtasPerSm);
            fold_scalar_kernel<__nv_bfloat16><<<grid, kThreads, 0, stream>>>(g, m, v, n, c.a, c.b);
        }
    }
    return cudaGetLastError();
}

cudaError_t launch_apply(float *w, float *m, float *v, size_t n, ApplyConstants c, int sm_count,
                         cudaStream_t stream, void *w_bf16_out) {
    __nv_bfloat16 *wb = static_cast<__nv_bfloat16 *>(w_bf16_out);
    if (n == 0) return cudaSuccess;
    constexpr int U = kApplyUnroll;
    const size_t n4 = n / 4;
    if (aligned(w, 16) && aligned(m, 16) && aligned(v, 16) && (!wb || aligned(wb, 8))) {
        unsigned grid = grid_for(n4, (size_t)kThreads * U, sm_count, kApplyCtasPerSm);
        if (wb)
            apply_vec_kernel<U, true><<<grid, kThreads, 0, stream>>>(w, m, v, wb, n4, n, c);
        else
            apply_vec_kernel<U, false><<<grid, kThreads, 0, stream>>>(w, m, v, nullptr, n4, n, c);
    } else {
        unsigned grid = grid_for(n, kThreads, sm_count, kCtasPerSm);
        apply_scalar_kernel<<<grid, kThreads, 0, stream>>>(w, m, v, wb, n, c);
    }
    return cudaGetLastError();
}

}  // namespace adama
