// Multi-tensor forms of the streaming kernels: one launch folds (or applies) up to 64
// parameter tensors, so that the hundreds of small tensors of a transformer (biases, norm
// scales) cost one launch per group instead of one each.  Same arithmetic as fold_apply.cu
// (Algorithm 2, inner loop body / "Update" + next decay); the table of pointers travels in
// the kernel's parameter space, no device memory is allocated.
#include <cuda_bf16.h>

#include "adama_device.cuh"

namespace adama {
namespace {

constexpr int kThreads = 256;
constexpr int kBlockElems = 4096;  // elements one CTA handles per step: 16 per thread

struct MultiTable {
    const void *g[kMultiMax];  // gradient (fold) -- unused by apply
    float *w[kMultiMax];       // weights (apply) -- unused by fold
    float *m[kMultiMax];
    float *v[kMultiMax];
    unsigned long long n[kMultiMax];
    unsigned block_start[kMultiMax + 1];  // prefix sum of ceil(n / kBlockElems)
    int count;
};
static_assert(sizeof(MultiTable) <= 4000, "table must fit the kernel parameter space");

__device__ __forceinline__ int find_tensor(const MultiTable &t, unsigned blk) {
    int lo = 0, hi = t.count;  // block_start[lo] <= blk < block_start[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (t.block_start[mid] <= blk) lo = mid;
        else hi = mid;
    }
    return lo;
}

__device__ __forceinline__ float widen(float g) { return g; }
__device__ __forceinline__ float widen(__nv_bfloat16 g) { return __bfloat162float(g); }

__device__ __forceinline__ void load4(const float *g, float (&x)[4]) {
    const float4 t = *reinterpret_cast<const float4 *>(g);
    x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16 *g, float (&x)[4]) {
    const uint2 t = *reinterpret_cast<const uint2 *>(g);
    x[0] = __uint_as_float(t.x << 16);
    x[1] = __uint_as_float(t.x & 0xffff0000u);
    x[2] = __uint_as_float(t.y << 16);
    x[3] = __uint_as_float(t.y & 0xffff0000u);
}

template <typename G>
__global__ void __launch_bounds__(kThreads)
fold_multi_kernel(const __grid_constant__ MultiTable tab, float a, float b) {
    const unsigned total = tab.block_start[tab.count];
    for (unsigned blk = blockIdx.x; blk < total; blk += gridDim.x) {
        const int t = find_tensor(tab, blk);
        const size_t base = (size_t)(blk - tab.block_start[t]) * kBlockElems;
        const size_t n = (size_t)tab.n[t];
        const size_t cnt = n - base < (size_t)kBlockElems ? n - base : (size_t)kBlockElems;
        const G *g = static_cast<const G *>(tab.g[t]) + base;
        float *m = tab.m[t] + base;
        float *v = tab.v[t] + base;
        const bool vec = ((reinterpret_cast<uintptr_t>(m) | reinterpret_cast<uintptr_t>(v)) & 15) == 0 &&
                         (reinterpret_cast<uintptr_t>(g) & (4 * sizeof(G) - 1)) == 0;
        if (vec) {
            const size_t c4 = cnt / 4;
            for (size_t i = threadIdx.x; i < c4; i += kThreads) {
                float x[4];
                load4(g + 4 * i, x);
                float4 mm = reinterpret_cast<float4 *>(m)[i], vv = reinterpret_cast<float4 *>(v)[i];
                fold1(x[0], mm.x, vv.x, a, b);
                fold1(x[1], mm.y, vv.y, a, b);
                fold1(x[2], mm.z, vv.z, a, b);
                fold1(x[3], mm.w, vv.w, a, b);
                reinterpret_cast<float4 *>(m)[i] = mm;
                reinterpret_cast<float4 *>(v)[i] = vv;
            }
            for (size_t i = c4 * 4 + threadIdx.x; i < cnt; i += kThreads) {
                fold1(widen(g[i]), m[i], v[i], a, b);
            }
        } else {
            for (size_t i = threadIdx.x; i < cnt; i += kThreads) {
                fold1(widen(g[i]), m[i], v[i], a, b);
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads)
apply_multi_kernel(const __grid_constant__ MultiTable tab, ApplyConstants c) {
    const unsigned total = tab.block_start[tab.count];
    for (unsigned blk = blockIdx.x; blk < total; blk += gridDim.x) {
        const int t = find_tensor(tab, blk);
        const size_t base = (size_t)(blk - tab.block_start[t]) * kBlockElems;
        const size_t n = (size_t)tab.n[t];
        const size_t cnt = n - base < (size_t)kBlockElems ? n - base : (size_t)kBlockElems;
        float *w = tab.w[t] + base;
        float *m = tab.m[t] + base;
        float *v = tab.v[t] + base;
        const bool vec = ((reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(m) |
                           reinterpret_cast<uintptr_t>(v)) & 15) == 0;
        size_t done = 0;
        if (vec) {
            const size_t c4 = cnt / 4;
            for (size_t i = threadIdx.x; i < c4; i += kThreads) {
                float4 ww = reinterpret_cast<float4 *>(w)[i], mm = reinterpret_cast<float4 *>(m)[i],
                       vv = reinterpret_cast<float4 *>(v)[i];
                apply1(ww.x, mm.x, vv.x, c);
                apply1(ww.y, mm.y, vv.y, c);
                apply1(ww.z, mm.z, vv.z, c);
                apply1(ww.w, mm.w, vv.w, c);
                reinterpret_cast<float4 *>(w)[i] = ww;
                reinterpret_cast<float4 *>(m)[i] = mm;
                reinterpret_cast<float4 *>(v)[i] = vv;
            }
            done = c4 * 4;
        }
        for (size_t i = done + threadIdx.x; i < cnt; i += kThreads) {
            float wi = w[i], mi = m[i], vi = v[i];
            apply1(wi, mi, vi, c);
            w[i] = wi;
            m[i] = mi;
            v[i] = vi;
        }
    }
}

// Fills block_start for tensors [first, first+count) and returns the number of blocks.
unsigned fill_blocks(MultiTable &tab, const size_t *n, int count) {
    unsigned acc = 0;
    for (int i = 0; i < count; ++i) {
        tab.n[i] = (unsigned long long)n[i];
        tab.block_start[i] = acc;
        acc += (unsigned)((n[i] + kBlockElems - 1) / kBlockElems);
    }
    tab.block_start[count] = acc;
    tab.count = count;
    return acc;
}

unsigned grid_for(unsigned blocks, int sm_count) {
    const unsigned cap = (unsigned)sm_count * 8u;
    return blocks < cap ? blocks : cap;
}

}  // namespace

cudaError_t launch_fold_multi(const void *const *g, adama_dtype gdt, float *const *m,
                              float *const *v, const size_t *n, int count, FoldConstants c,
                              int sm_count, cudaStream_t stream) {
    MultiTable tab;
    for (int i = 0; i < count; ++i) {
        tab.g[i] = g[i];
        tab.w[i] = nullptr;
        tab.m[i] = m[i];
        tab.v[i] = v[i];
    }
    const unsigned blocks = fill_blocks(tab, n, count);
    if (blocks == 0) return cudaSuccess;
    const unsigned grid = grid_for(blocks, sm_count);
    if (gdt == ADAMA_F32)
        fold_multi_kernel<float><<<grid, kThreads, 0, stream>>>(tab, c.a, c.b);
    else
        fold_multi_kernel<__nv_bfloat16><<<grid, kThreads, 0, stream>>>(tab, c.a, c.b);
    return cudaGetLastError();
}

cudaError_t launch_apply_multi(float *const *w, float *const *m, float *const *v, const size_t *n,
                               int count, ApplyConstants c, int sm_count, cudaStream_t stream) {
    MultiTable tab;
    for (int i = 0; i < count; ++i) {
        tab.g[i] = nullptr;
        tab.w[i] = w[i];
        tab.m[i] = m[i];
        tab.v[i] = v[i];
    }
    const unsigned blocks = fill_blocks(tab, n, count);
    if (blocks == 0) return cudaSuccess;
    apply_multi_kernel<<<grid_for(blocks, sm_count), kThreads, 0, stream>>>(tab, c);
    return cudaGetLastError();
}

}  // namespace adama
