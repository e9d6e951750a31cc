// State-sharded update with the exchange fused in: reduce-scatter of m and v, the update of
// the owner's shard of w, and the all-gather of w, as ONE kernel over peer-mapped buffers
// (NVLink / NVSwitch peer access: plain 128-bit loads and stores, no multicast, no waiting
// inside the kernel; the loads of up to 8 peers are issued together so that their round trips
// overlap).  Rank r's launch touches only shard r of every rank's w, m and v:
//   S_m = sum_q m_q[shard r],  S_v = sum_q v_q[shard r]            (rank order: deterministic)
//   w_new = update(w_r, S_m / R, S_v / R^2)                        (Algorithm 2 "Update" on the
//                                                                   averaged states, Eqs. 6-7)
//   m_r[shard r] = beta1*S_m, v_r[shard r] = beta2*S_v;  m_q = v_q = 0 on that shard for q != r
//   w_q[shard r] = w_new for every q
// The ranks must have finished folding before any of these launches starts and must not fold
// again before all of them have finished; that ordering is the caller's (a barrier on the
// host or between streams), so the kernel itself never waits for a peer.
#include "adama_device.cuh"

namespace adama {
namespace {

constexpr int kThreads = 256;
constexpr int kPeerBatch = 8;  // peers whose m, v loads are in flight together (64 data registers)

struct PeerTable {
    float *w[kMaxPeers];
    float *m[kMaxPeers];
    float *v[kMaxPeers];
    int world;
    int rank;
};

__device__ __forceinline__ float4 ld4(const float *p) {
    float4 r;
    asm volatile("ld.global.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w)
                 : "l"(p));
    return r;
}
__device__ __forceinline__ void st4(float *p, float4 x) {
    asm volatile("st.global.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(p), "f"(x.x), "f"(x.y), "f"(x.z),
                 "f"(x.w)
                 : "memory");
}
__global__ void __launch_bounds__(kThreads)
apply_sharded_peers_kernel(const __grid_constant__ PeerTable tab, size_t lo4, size_t n4,
                           ApplyConstants c) {
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < n4;
         i += (size_t)gridDim.x * kThreads) {
        const size_t e = (lo4 + i) * 4;
        // All loads of a batch of peers are issued before the first add, so that their NVLink
        // round trips overlap; the adds then run in rank order (deterministic, and the same
        // sums as a serial loop over the peers).
        float4 sm = zero, sv = zero;
        float4 w = ld4(tab.w[tab.rank] + e);
        for (int q0 = 0; q0 < tab.world; q0 += kPeerBatch) {
            float4 a[kPeerBatch], b[kPeerBatch];
#pragma unroll
            for (int j = 0; j < kPeerBatch; ++j)
                if (q0 + j < tab.world) {
                    a[j] = ld4(tab.m[q0 + j] + e);
                    b[j] = ld4(tab.v[q0 + j] + e);
                }
#pragma unroll
            for (int j = 0; j < kPeerBatch; ++j)
                if (q0 + j < tab.world) {
                    sm.x += a[j].x; sm.y += a[j].y; sm.z += a[j].z; sm.w += a[j].w;
                    sv.x += b[j].x; sv.y += b[j].y; sv.z += b[j].z; sv.w += b[j].w;
                }
        }
        apply1(w.x, sm.x, sv.x, c);
        apply1(w.y, sm.y, sv.y, c);
        apply1(w.z, sm.z, sv.z, c);
        apply1(w.w, sm.w, sv.w, c);
        for (int q = 0; q < tab.world; ++q) {
            st4(tab.w[q] + e, w);
            st4(tab.m[q] + e, q == tab.rank ? sm : zero);
            st4(tab.v[q] + e, q == tab.rank ? sv : zero);
        }
    }
}

}  // namespace

cudaError_t launch_apply_sharded_peers(float *const *w, float *const *m, float *const *v, int world,
                                       int rank, size_t n, ApplyConstants c, int sm_count,
                                       cudaStream_t stream) {
    PeerTable tab;
    for (int q = 0; q < world; ++q) {
        tab.w[q] = w[q];
        tab.m[q] = m[q];
        tab.v[q] = v[q];
    }
    tab.world = world;
    tab.rank = rank;
    const size_t shard4 = n / 4 / (size_t)world;
    if (shard4 == 0) return cudaSuccess;
    size_t need = (shard4 + kThreads - 1) / kThreads;
    const size_t cap = (size_t)sm_count * 4;
    const unsigned grid = (unsigned)(need < cap ? need : cap);
    apply_sharded_peers_kernel<<<grid, kThreads, 0, stream>>>(tab, shard4 * (size_t)rank, shard4, c);
    return cudaGetLastError();
}

}  // namespace adama
