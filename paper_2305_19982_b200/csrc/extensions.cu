// Two additions on the skeleton of the streaming kernels:
//  * SGD with momentum folded micro-batch by micro-batch (the paper's Discussion: other momentum
//    optimizers can take the same accumulation): buf += g/N per micro-batch, then
//    w -= lr*buf and buf *= mu for the next mini-batch in one pass;
//  * the coefficient sqrt(v_hat)/sqrt(v_hat') of Section 4.1 between AdamA's and standard Adam's
//    adaptive scaling: mean and range over the elements, with Adam's second moment v' carried
//    in a buffer of its own and the mini-batch gradient sum recovered from the change of m.
#include <cuda_bf16.h>
#include <math.h>

#include "adama_internal.h"
#include "stream_access.cuh"

namespace adama {
namespace {

// Unroll factors from a sweep at 335 M elements on B200 (GB/s): sgdm fold 8/12/16/24 -> 5359/5731/
// 5565/5753; sgdm apply 8/10/12/16 -> 6169/6077/6043/6015; coefficient 3/4/6/8 -> 4322/4669/5105/5366.
constexpr int kThreads = 256;
constexpr int kSgdmFoldUnroll = 12;   // {g, buf} 128-bit groups in flight per thread
constexpr int kSgdmApplyUnroll = 8;   // {w, buf}
constexpr int kCoefUnroll = 8;        // {m, m_begin, v, v_adam}

template <typename G, int UNROLL>
__global__ void __launch_bounds__(kThreads, 1)
sgdm_fold_vec_kernel(const G *__restrict__ grad, float *__restrict__ buf, size_t n4, size_t n,
                     float inv_n) {
    float4 *b4 = reinterpret_cast<float4 *>(buf);
    const size_t span = (size_t)kThreads * UNROLL;
    for (size_t base = (size_t)blockIdx.x * span; base < n4; base += (size_t)gridDim.x * span) {
        Grad4 g[UNROLL];
        float4 bb[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            size_t i = base + (size_t)u * kThreads + threadIdx.x;
            if (i < n4) {
                g[u] = load_grad4(grad, i);
                bb[u] = ld_stream(b4 + i);
            }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            size_t i = base + (size_t)u * kThreads + threadIdx.x;
            if (i < n4) {
                bb[u].x = fmaf(inv_n, g[u].x, bb[u].x);
                bb[u].y = fmaf(inv_n, g[u].y, bb[u].y);
                bb[u].z = fmaf(inv_n, g[u].z, bb[u].z);
                bb[u].w = fmaf(inv_n, g[u].w, bb[u].w);
                st_stream(b4 + i, bb[u]);
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x < (unsigned)(n - n4 * 4)) {
        size_t i = n4 * 4 + threadIdx.x;
        buf[i] = fmaf(inv_n, widen(grad[i]), buf[i]);
    }
}

template <typename G>
__global__ void __launch_bounds__(kThreads)
sgdm_fold_scalar_kernel(const G *__restrict__ grad, float *__restrict__ buf, size_t n, float inv_n) {
    for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < n;
         i += (size_t)gridDim.x * kThreads)
        buf[i] = fmaf(inv_n, widen(grad[i]), buf[i]);
}

// w -= lr*buf; buf *= mu (mu = hi + lo, one rounding: see the decay of the Adam moments)
__device__ __forceinline__ void sgdm_apply1(float &w, float &b, float lr, float mu_hi, float mu_lo) {
    w = fmaf(-lr, b, w);
    b = fmaf(b, mu_hi, b * mu_lo);
}

template <int UNROLL>
__global__ void __launch_bounds__(kThreads, 1)
sgdm_apply_vec_kernel(float *__restrict__ w, float *__restrict__ buf, size_t n4, size_t n, float lr,
                      float mu_hi, float mu_lo) {
    float4 *w4 = reinterpret_cast<float4 *>(w);
    float4 *b4 = reinterpret_cast<float4 *>(buf);
    const size_t span = (size_t)kThreads * UNROLL;
    for (size_t base = (size_t)blockIdx.x * span; base < n4; base += (size_t)gridDim.x * span) {
        float4 ww[UNROLL], bb[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            size_t i = base + (size_t)u * kThreads + threadIdx.x;
            if (i < n4) {
                ww[u] = ld_stream(w4 + i);
                bb[u] = ld_stream(b4 + i);
            }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            size_t i = base + (size_t)u * kThreads + threadIdx.x;
            if (i < n4) {
                sgdm_apply1(ww[u].x, bb[u].x, lr, mu_hi, mu_lo);
                sgdm_apply1(ww[u].y, bb[u].y, lr, mu_hi, mu_lo);
                sgdm_apply1(ww[u].z, bb[u].z, lr, mu_hi, mu_lo);
                sgdm_apply1(ww[u].w, bb[u].w, lr, mu_hi, mu_lo);
                st_stream(w4 + i, ww[u]);
                st_stream(b4 + i, bb[u]);
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x < (unsigned)(n - n4 * 4)) {
        size_t i = n4 * 4 + threadIdx.x;
        float wi = w[i], bi = buf[i];
        sgdm_apply1(wi, bi, lr, mu_hi, mu_lo);
        w[i] = wi;
        buf[i] = bi;
    }
}

__global__ void __launch_bounds__(kThreads)
sgdm_apply_scalar_kernel(float *__restrict__ w, float *__restrict__ buf, size_t n, float lr,
                         float mu_hi, float mu_lo) {
    for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < n;
         i += (size_t)gridDim.x * kThreads) {
        float wi = w[i], bi = buf[i];
        sgdm_apply1(wi, bi, lr, mu_hi, mu_lo);
        w[i] = wi;
        buf[i] = bi;
    }
}

// ---- coefficient statistics -----------------------------------------------------------------

struct CoefAcc {
    double sum;
    float lo, hi;
    unsigned long long count;
};

// One element: Adam's second moment of this mini-batch from the change of m, the coefficient,
// and the stored v' decayed for the next mini-batch.
//   d = m - m_begin = (1-beta1) * sum_i g_i     =>  (1-beta2) (sum_i g_i)^2 = k * d^2
__device__ __forceinline__ void coef1(float m, float m0, float v, float &va, const CoefConstants &c,
                                      float &s4, CoefAcc &acc) {
    const float d = m - m0;
    const float va_t = fmaf(c.k * d, d, va);
    if (va_t > 0.f) {
        const float co = sqrtf(v / va_t);  // the bias corrections 1/(1-beta2^t) cancel
        s4 += co;
        acc.lo = fminf(acc.lo, co);
        acc.hi = fmaxf(acc.hi, co);
        acc.count += 1;
    }
    va = fmaf(va_t, c.beta2_hi, va_t * c.beta2_lo);
}

// stats[0] += sum of c, stats[1] = min, stats[2] = max, stats[3] += count (all doubles; the
// coefficients are >= 0, so min and max order like their bit patterns)
__device__ __forceinline__ void coef_commit(const CoefAcc &mine, double *stats) {
    __shared__ double s_sum[kThreads / 32];
    __shared__ float s_lo[kThreads / 32], s_hi[kThreads / 32];
    __shared__ unsigned long long s_cnt[kThreads / 32];
    double sum = mine.sum;
    float lo = mine.lo, hi = mine.hi;
    unsigned long long cnt = mine.count;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        sum += __shfl_xor_sync(0xffffffffu, sum, off);
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, off));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, off));
        cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) {
        s_sum[warp] = sum;
        s_lo[warp] = lo;
        s_hi[warp] = hi;
        s_cnt[warp] = cnt;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kThreads / 32; ++w) {
            sum += s_sum[w];
            lo = fminf(lo, s_lo[w]);
            hi = fmaxf(hi, s_hi[w]);
            cnt += s_cnt[w];
        }
        if (cnt) {
            atomicAdd(stats + 0, sum);
            atomicMin(reinterpret_cast<unsigned long long *>(stats + 1),
                      (unsigned long long)__double_as_longlong((double)lo));
            atomicMax(reinterpret_cast<unsigned long long *>(stats + 2),
                      (unsigned long long)__double_as_longlong((double)hi));
            atomicAdd(stats + 3, (double)cnt);
        }
    }
}

__global__ void coef_init_kernel(double *stats) {
    stats[0] = 0.0;
    stats[1] = INFINITY;
    stats[2] = 0.0;
    stats[3] = 0.0;
}

template <int UNROLL, bool HAS_BEGIN>
__global__ void __launch_bounds__(kThreads, 1)
coef_vec_kernel(const float *__restrict__ m, const float *__restrict__ m_begin,
                const float *__restrict__ v, float *__restrict__ v_adam, size_t n4, size_t n,
                CoefConstants c, double *__restrict__ stats) {
    const float4 *m4 = reinterpret_cast<const float4 *>(m);
    const float4 *m04 = reinterpret_cast<const float4 *>(m_begin);
    const float4 *v4 = reinterpret_cast<const float4 *>(v);
    float4 *va4 = reinterpret_cast<float4 *>(v_adam);
    CoefAcc acc = {0.0, INFINITY, 0.f, 0ull};
    const size_t span = (size_t)kThreads * UNROLL;
    for (size_t base = (size_t)blockIdx.x * span; base < n4; base += (size_t)gridDim.x * span) {
        float4 mm[UNROLL], m0[UNROLL], vv[UNROLL], va[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            size_t i = base + (size_t)u * kThreads + threadIdx.x;
            if (i < n4) {
                mm[u] = ld_stream_ro(m4 + i);
                m0[u] = HAS_BEGIN ? ld_stream_ro(m04 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                vv[u] = ld_stream_ro(v4 + i);
                va[u] = ld_stream(va4 + i);
            }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            size_t i = base + (size_t)u * kThreads + threadIdx.x;
            if (i < n4) {
                float s4 = 0.f;
                coef1(mm[u].x, m0[u].x, vv[u].x, va[u].x, c, s4, acc);
                coef1(mm[u].y, m0[u].y, vv[u].y, va[u].y, c, s4, acc);
                coef1(mm[u].z, m0[u].z, vv[u].z, va[u].z, c, s4, acc);
                coef1(mm[u].w, m0[u].w, vv[u].w, va[u].w, c, s4, acc);
                acc.sum += (double)s4;
                st_stream(va4 + i, va[u]);
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x < (unsigned)(n - n4 * 4)) {
        size_t i = n4 * 4 + threadIdx.x;
        float s4 = 0.f, va = v_adam[i];
        coef1(m[i], HAS_BEGIN ? m_begin[i] : 0.f, v[i], va, c, s4, acc);
        acc.sum += (double)s4;
        v_adam[i] = va;
    }
    coef_commit(acc, stats);
}

template <bool HAS_BEGIN>
__global__ void __launch_bounds__(kThreads)
coef_scalar_kernel(const float *__restrict__ m, const float *__restrict__ m_begin,
                   const float *__restrict__ v, float *__restrict__ v_adam, size_t n,
                   CoefConstants c, double *__restrict__ stats) {
    CoefAcc acc = {0.0, INFINITY, 0.f, 0ull};
    for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < n;
         i += (size_t)gridDim.x * kThreads) {
        float s4 = 0.f, va = v_adam[i];
        coef1(m[i], HAS_BEGIN ? m_begin[i] : 0.f, v[i], va, c, s4, acc);
        acc.sum += (double)s4;
        v_adam[i] = va;
    }
    coef_commit(acc, stats);
}

}  // namespace

cudaError_t launch_sgdm_fold(const void *grad, adama_dtype gdt, float *buf, size_t n, float inv_n,
                             int sm_count, cudaStream_t stream) {
    if (n == 0) return cudaSuccess;
    constexpr int U = kSgdmFoldUnroll;
    const size_t n4 = n / 4;
    const bool vec = aligned(buf, 16) && aligned(grad, gdt == ADAMA_F32 ? 16 : 8);
    const unsigned grid = vec ? grid_for(n4, (size_t)kThreads * U, sm_count, 1)
                              : grid_for(n, kThreads, sm_count, 4);
    if (gdt == ADAMA_F32) {
        const float *g = static_cast<const float *>(grad);
        if (vec)
            sgdm_fold_vec_kernel<float, U><<<grid, kThreads, 0, stream>>>(g, buf, n4, n, inv_n);
        else
            sgdm_fold_scalar_kernel<float><<<grid, kThreads, 0, stream>>>(g, buf, n, inv_n);
    } else {
        const __nv_bfloat16 *g = static_cast<const __nv_bfloat16 *>(grad);
        if (vec)
            sgdm_fold_vec_kernel<__nv_bfloat16, U><<<grid, kThreads, 0, stream>>>(g, buf, n4, n, inv_n);
        else
            sgdm_fold_scalar_kernel<__nv_bfloat16><<<grid, kThreads, 0, stream>>>(g, buf, n, inv_n);
    }
    return cudaGetLastError();
}

cudaError_t launch_sgdm_apply(float *w, float *buf, size_t n, float lr, float mu_hi, float mu_lo,
                              int sm_count, cudaStream_t stream) {
    if (n == 0) return cudaSuccess;
    constexpr int U = kSgdmApplyUnroll;
    const size_t n4 = n / 4;
    if (aligned(w, 16) && aligned(buf, 16)) {
        const unsigned grid = grid_for(n4, (size_t)kThreads * U, sm_count, 1);
        sgdm_apply_vec_kernel<U><<<grid, kThreads, 0, stream>>>(w, buf, n4, n, lr, mu_hi, mu_lo);
    } else {
        const unsigned grid = grid_for(n, kThreads, sm_count, 4);
        sgdm_apply_scalar_kernel<<<grid, kThreads, 0, stream>>>(w, buf, n, lr, mu_hi, mu_lo);
    }
    return cudaGetLastError();
}

cudaError_t launch_coefficient_stats(const float *m, const float *m_begin, const float *v,
                                     float *v_adam, size_t n, CoefConstants c, double *stats,
                                     int sm_count, cudaStream_t stream) {
    coef_init_kernel<<<1, 1, 0, stream>>>(stats);
    if (n == 0) return cudaGetLastError();
    constexpr int U = kCoefUnroll;
    const size_t n4 = n / 4;
    const bool vec = aligned(m, 16) && aligned(v, 16) && aligned(v_adam, 16) &&
                     (!m_begin || aligned(m_begin, 16));
    if (vec) {
        const unsigned grid = grid_for(n4, (size_t)kThreads * U, sm_count, 1);
        if (m_begin)
            coef_vec_kernel<U, true><<<grid, kThreads, 0, stream>>>(m, m_begin, v, v_adam, n4, n, c, stats);
        else
            coef_vec_kernel<U, false><<<grid, kThreads, 0, stream>>>(m, nullptr, v, v_adam, n4, n, c, stats);
    } else {
        const unsigned grid = grid_for(n, kThreads, sm_count, 4);
        if (m_begin)
            coef_scalar_kernel<true><<<grid, kThreads, 0, stream>>>(m, m_begin, v, v_adam, n, c, stats);
        else
            coef_scalar_kernel<false><<<grid, kThreads, 0, stream>>>(m, nullptr, v, v_adam, n, c, stats);
    }
    return cudaGetLastError();
}

}  // namespace adama
