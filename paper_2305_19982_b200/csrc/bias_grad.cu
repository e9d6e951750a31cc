// Bias gradient of a linear layer folded into its moments:
//     g[q]  = sum_tau dY[tau, q]                     (raw micro-batch gradient of the bias)
//     m[q] += a*g[q];  v[q] += b*g[q]^2              (Algorithm 2, inner loop body)
// The token sum must be complete before it is squared, so the partial sums of the CTAs that
// share a column slab are combined on-chip: a cluster of 8 CTAs splits the tokens, each leaves
// its 256 partial sums in shared memory, and the cluster's first CTA adds the eight vectors
// through distributed shared memory, in rank order (deterministic), and folds.  One pass over
// dY (2*tokens*d_out bytes), nothing written but m and v.
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include "adama_internal.h"

namespace cg = cooperative_groups;

namespace adama {
namespace {

constexpr int kColsPerThread = 8;                  // 8 bf16 = one 16-byte load
constexpr int kSlabCols = 32 * kColsPerThread;     // 256 columns per cluster
constexpr int kRowLanes = 16;                      // rows read concurrently by one CTA
constexpr int kUnroll = 8;                         // independent 16-byte loads in flight per thread
constexpr int kThreads = 32 * kRowLanes;
constexpr int kClusterSize = 8;  // CTAs that split the tokens of one slab

__global__ void __launch_bounds__(kThreads)
bias_grad_fold_kernel(const __nv_bfloat16 *__restrict__ dY, int tokens, int d_out, long long ldy,
                      float *__restrict__ m, float *__restrict__ v, float a, float b) {
    __shared__ float part[kRowLanes][kSlabCols];
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned rank = cluster.block_rank();
    const int slab = blockIdx.x / kClusterSize;
    const int cgp = threadIdx.x & 31;  // column group: 8 columns
    const int rl = threadIdx.x >> 5;   // row lane
    const int col = slab * kSlabCols + cgp * kColsPerThread;
    // this CTA's share of the tokens
    const int per = (tokens + kClusterSize - 1) / kClusterSize;
    const int t0 = (int)rank * per;
    const int t1 = t0 + per < tokens ? t0 + per : tokens;

    float acc[kColsPerThread];
#pragma unroll
    for (int e = 0; e < kColsPerThread; ++e) acc[e] = 0.f;
    if (col + kColsPerThread <= d_out) {
        int tau = t0 + rl;
        for (; tau + (kUnroll - 1) * kRowLanes < t1; tau += kUnroll * kRowLanes) {
            uint4 x[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u)
                x[u] = *reinterpret_cast<const uint4 *>(dY + (long long)(tau + u * kRowLanes) * ldy + col);
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const unsigned wds[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    acc[2 * k] += __uint_as_float(wds[k] << 16);
                    acc[2 * k + 1] += __uint_as_float(wds[k] & 0xffff0000u);
                }
            }
        }
        for (; tau < t1; tau += kRowLanes) {
            const uint4 x = *reinterpret_cast<const uint4 *>(dY + (long long)tau * ldy + col);
            const unsigned wds[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                acc[2 * k] += __uint_as_float(wds[k] << 16);
                acc[2 * k + 1] += __uint_as_float(wds[k] & 0xffff0000u);
            }
        }
    } else {
        for (int tau = t0 + rl; tau < t1; tau += kRowLanes)
            for (int e = 0; e < kColsPerThread; ++e)
                if (col + e < d_out) acc[e] += __bfloat162float(dY[(long long)tau * ldy + col + e]);
    }
#pragma unroll
    for (int e = 0; e < kColsPerThread; ++e) part[rl][cgp * kColsPerThread + e] = acc[e];
    __syncthreads();
    // row lanes -> one vector per CTA, kept in part[0]
    if (threadIdx.x < kSlabCols) {
        float s = 0.f;
#pragma unroll
        for (int r = 0; r < kRowLanes; ++r) s += part[r][threadIdx.x];
        part[0][threadIdx.x] = s;
    }
    cluster.sync();  // every CTA's vector is in place
    if (rank == 0 && threadIdx.x < kSlabCols) {
        const int q = slab * kSlabCols + threadIdx.x;
        if (q < d_out) {
            float g = 0.f;
            for (unsigned r = 0; r < (unsigned)kClusterSize; ++r)
                g += cluster.map_shared_rank(&part[0][0], r)[threadIdx.x];
            m[q] = fmaf(a, g, m[q]);
            v[q] = fmaf(b * g, g, v[q]);
        }
    }
    cluster.sync();  // no CTA leaves while its shared memory may still be read
}

}  // namespace

cudaError_t launch_bias_grad_fold(const void *dY, int tokens, int d_out, int64_t ldy, float *m,
                                  float *v, FoldConstants c, cudaStream_t stream) {
    const int slabs = (d_out + kSlabCols - 1) / kSlabCols;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(slabs * kClusterSize), 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kClusterSize;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, bias_grad_fold_kernel, static_cast<const __nv_bfloat16 *>(dY),
                              tokens, d_out, (long long)ldy, m, v, c.a, c.b);
}

}  // namespace adama
