// Fused linear-layer weight gradient + AdamA fold for sm_100a.
//
//   G[p,q]  = sum_tau X[tau,p] * dY[tau,q]          (bf16 x bf16 -> fp32, tcgen05.mma)
//   m[p,q] += a*G[p,q];   v[p,q] += b*G[p,q]^2       (Algorithm 2, inner loop body)
//
// G lives only as an accumulator tile in tensor memory.  The epilogue issues the
// coalesced 128-bit loads of the matching m chunk first, reads the accumulator
// chunk with tcgen05.ld while they are in flight, turns it from "one row per thread"
// into "128 contiguous bytes per quarter-warp" through a swizzled shared-memory
// buffer, writes fma(a, G, m) back with 128-bit stores and hands (b*G)*G to the L2 as
// a reduction into v (red.global.add.v4.f32).  What bounds the main loop is the SM's
// inbound port from the L2 (about 118 GB/s per SM measured with TMA loads alone): a
// 256x256 pair tile needs 512 bytes of operands per token and SM, and the m, v reads of
// the overlapped epilogue come through the same port.  Sending v's half of the state
// traffic as reductions takes it off that port (config-3 call 122 -> 117 us); sending
// m's half too was measured slower (127 us): the L2's reduction rate then holds up the
// operand loads.
//
// Persistent kernel, 192 or 320 threads per CTA, CTAs working in pairs (a cluster of two on
// the two SMs of a TPC, tcgen05 cta_group::2): a pair owns a 256x256 output tile,
// each CTA its 128 rows.  Per 64-token stage a CTA loads its own 128 rows of X^T and
// only HALF of the dY tile (128 of the 256 columns); the tensor cores of both SMs
// read both halves.  That is 64 bytes of operands per tensor-core clock and SM
// instead of 96 for a lone 128x256 tile, and leaves room for a 6-stage ring.
//   warp 0      TMA producer: operand tiles -> shared-memory ring (both CTAs)
//   warp 1      MMA issuer (one thread of the pair's first CTA) + TMEM allocation
//   warps 2..   epilogue: one or two warps per TMEM lane quarter (4 or 8 warps, chosen per
//               launch; with two, each takes half of the tile's columns), in both CTAs
// The 512 TMEM columns hold two 128x256 fp32 accumulators per CTA, so the epilogue of
// tile i overlaps the main loop of tile i+1.
//   optional    two more warps that sum dY's columns into the bias moments (see the bias branch)
// Calls of up to 2048 tokens run a second instance with a "staged" epilogue (see STAGED_RING):
// 4 drain warps copy the accumulator to shared memory part by part, 8 streaming warps fold
// the parts into m and v; the ring has 5 stages there.
//
// What bounds the main loop is the round trip of a ring stage, not the tensor core: a 2-CTA
// tcgen05.mma of M = 256, N = 256, K = 16 takes 128 clocks (64 at N = 128), but a stage is held
// from its TMA issue until tcgen05.commit reports its MMAs retired -- load latency + 512
// clocks of MMAs + about 1600 clocks of commit latency + two wake-ups, some 3500 clocks against
// the 6 x 512 that six stages cover.  Hence: every stage counts, a 128-column tile runs its
// main loop no faster than a 256-column one (only 256 x 256 tiles are efficient), and the
// barrier probes carry a suspend-time hint so that waiters wake without delay.
//
// Operand layout.  The contraction runs over tokens, the strided dimension of both
// row-major inputs, so both operands are "MN-major": a TMA box of 64 features x 64
// tokens lands as 64 rows of 128 bytes (one token per row) under the 128-byte
// swizzle.  The shared-memory matrix descriptor states: 8-token groups 1024 bytes
// apart (stride byte offset), 64-feature groups one box (8192 bytes) apart (leading
// byte offset).
//
// Synchronisation of a pair: the first CTA's "full" barrier of a stage counts the
// bytes of both CTAs' loads; when the MMAs that read a stage retire, tcgen05.commit
// arrives on the "empty" barrier of each CTA; the same for accumulator-full; the
// epilogue warps of both CTAs arrive on the first CTA's accumulator-empty barrier.  No load uses cluster multicast.
//
// Every wait on an mbarrier is bounded (2 s of %globaltimer); on expiry the kernel
// records a code in the status block, all roles drain and leave, TMEM is freed.
#include <cuda.h>
#include <cuda_bf16.h>

#include <mutex>

#include "adama_internal.h"

namespace adama {
namespace {

constexpr int RING_STAGES = 6;  // shared-memory ring depth of the direct-epilogue instance
constexpr int BN = 256;     // tile columns (d_out direction) = UMMA N
constexpr int BK = 64;      // tokens per pipeline stage
constexpr int UMMA_K = 16;  // tokens per tcgen05.mma (bf16)
constexpr int GROUP = 64;   // features per 128-byte swizzled row
constexpr int BOX_BYTES = GROUP * BK * 2;               // 8192
constexpr int EPI_COLS = 32;                            // fp32 columns per epilogue chunk (128 B)
constexpr int EPI_ROWS = 32;                            // one TMEM lane quarter
constexpr int EPI_BUF_BYTES = EPI_ROWS * EPI_COLS * 4;  // 4096: one transposition buffer per warp
// Epilogue warps: 4 (one per TMEM lane quarter) or 8 (two per quarter, each half of the tile's
// columns), chosen per launch through the block size.  Measured: when tiles queue up behind
// each other 4 warps disturb the overlapped main loop less (4096x11008: 274 vs 279 us); when
// every CTA pair has a single tile its epilogue is fully exposed and 8 warps finish it sooner
// (1600x1600: 41.8 vs 43.8 us).
constexpr int MAX_EPI_WARPS = 8;
constexpr int EPI_BYTES = MAX_EPI_WARPS * EPI_BUF_BYTES;
constexpr int MAX_THREADS = 32 * (2 + MAX_EPI_WARPS + 2);  // + the two optional bias warps
constexpr int TMEM_COLS = 512;
constexpr int ACC_STAGES = 2;
constexpr int MAX_STAGES = 12;
constexpr int SMEM_BAR_BYTES = 512;
constexpr int BIAS_UNROLL = 8;  // 16-byte loads in flight per thread of a bias warp
constexpr int BIAS_WARPS = 2;
constexpr int SMEM_BIAS_BYTES = BIAS_WARPS * 32 * 4;

// Staged epilogue (calls of few tokens, where the m, v traffic bounds the call): the accumulator
// tile is first copied into shared memory, part by part (128 rows x PART_COLS fp32, two part
// buffers, the rest of the shared memory stays with the ring), and separate streaming warps
// fold the parts into m and v.
constexpr int PART_COLS = 64;                           // columns of one part of the tile copy
constexpr int PART_BYTES = 128 * PART_COLS * 4;         // 128 rows: 32 KB (64 columns) or 64 KB (128)
constexpr int STAGED_RING = (224 * 1024 - 2 * PART_BYTES) / (32 * 1024);  // 5 or 3 stages
constexpr int STAGED_DRAIN_WARPS = 4;   // tensor memory -> shared memory, one per lane quarter
constexpr int STAGED_STREAM_WARPS = 8;  // shared memory -> m, v (16 rows of the tile each)
constexpr int G_TILE_BYTES = 2 * PART_BYTES;  // two parts: one is filled while the other is folded
constexpr int STAGED_THREADS = 32 * (2 + STAGED_DRAIN_WARPS + STAGED_STREAM_WARPS + BIAS_WARPS);

constexpr int CTAS = 2;  // CTAs cooperating on one tile (tcgen05 cta_group::2)

// Per-variant geometry (STAGED: the short-call instance with the staged epilogue).
template <bool STAGED = false>
struct Geo {
    static constexpr int ROWS_PER_CTA = 128;                 // TMEM lanes
    static constexpr int TILE_M = ROWS_PER_CTA * CTAS;       // UMMA M
    static constexpr int B_COLS_PER_CTA = BN / CTAS;         // dY columns this CTA stages
    static constexpr int A_BOXES = ROWS_PER_CTA / GROUP;     // 2
    static constexpr int B_BOXES = B_COLS_PER_CTA / GROUP;   // 4 or 2
    static constexpr int A_STAGE_BYTES = A_BOXES * BOX_BYTES;
    static constexpr int B_STAGE_BYTES = B_BOXES * BOX_BYTES;
    static constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;  // 48 KB or 32 KB
    static constexpr int STAGES =
        STAGED ? STAGED_RING : RING_STAGES;
    static constexpr int SMEM_EPI_OFF = STAGES * STAGE_BYTES;
    static constexpr int SMEM_BAR_OFF = SMEM_EPI_OFF + (STAGED ? G_TILE_BYTES : EPI_BYTES);
    static constexpr int SMEM_BIAS_OFF = SMEM_BAR_OFF + SMEM_BAR_BYTES;
    static constexpr int SMEM_BYTES = SMEM_BIAS_OFF + SMEM_BIAS_BYTES + 1024;  // + alignment slack
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
    static_assert(STAGES <= MAX_STAGES, "barrier block");
    // tcgen05 instruction descriptor, kind::f16: fp32 accumulate, bf16 A and B, both
    // MN-major, M = 128 per participating CTA; N (bits 17..22, in units of 8) is added
    // per work item.
    static constexpr uint32_t INSTR_DESC_NO_N = (1u << 4)     // D format: f32
                                                | (1u << 7)   // A format: bf16
                                                | (1u << 10)  // B format: bf16
                                                | (1u << 15)  // A is MN-major
                                                | (1u << 16)  // B is MN-major
                                                | ((uint32_t)(TILE_M >> 4) << 24);
};

constexpr unsigned long long kDrainLimitNs = 20000000ull;   // 20 ms

// ---- PTX wrappers --------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ unsigned long long globaltimer() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of `addr` (a shared::cta address) in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;"
                 ::: "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// arrive on a barrier given by its shared::cluster address (own CTA or the partner)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
// One probe of a barrier phase.  The explicit suspend-time hint matters: with it a thread that
// waits on a barrier is back ~250 clocks sooner after the phase completes than with the default
// time limit, and both the producer (waiting for a free stage) and the MMA issuer (waiting for a
// full one) sit on the critical path of the operand ring (config-3 call 120.9 -> 118.8 us,
// 4096x11008 305 -> 300 us; any hint from 32 ns to 2 us measured the same).
constexpr uint32_t kSuspendHintNs = 64;
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(kSuspendHintNs)
        : "memory");
    return ok != 0;
}
// Bounded wait: false if `limit_ns` passed or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          unsigned long long limit_ns) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = globaltimer();
    for (uint32_t spins = 1;; ++spins) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spins & 0x3f) == 0) {
            if (*abort_flag) return false;
            if (globaltimer() - t0 > limit_ns) return false;
        }
    }
}
// TMA tile load into this CTA's shared memory; `bar` is a shared::cluster address and may
// name the partner CTA's barrier.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
// Same, through a 3-D view {64 features, tokens, 64-feature groups}: one operation brings
// several 64-feature groups (boxes of 8192 bytes, one after the other in shared memory).
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int tok, int grp,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
        "l"(map), "r"(0), "r"(tok), "r"(grp), "r"(bar)
        : "memory");
}
// Programmatic dependent launch.  grid_dependency_wait: returns once the kernel launched before
// this one in the stream has completed and its writes are visible (at once if this launch was
// not made programmatic).  grid_launch_dependents: the next kernel in the stream, if it was
// launched programmatic, may start its CTAs as soon as this grid's CTAs have all got here or
// exited and an SM is free.
__device__ __forceinline__ void grid_dependency_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
__device__ __forceinline__ void grid_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// Arrive on `cluster_bar` (shared::cluster address) once all MMAs issued so far by this
// thread have retired.
__device__ __forceinline__ void tc_commit(uint32_t cluster_bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                     cluster_bar)
                 : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b,
                                       uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem),
                 "n"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "n"(TMEM_COLS)
                 : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread i receives TMEM lane (base lane + i).
__device__ __forceinline__ void tc_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
          "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
          "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]),
          "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]),
          "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld() {
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ float4 ld_shared_v4(uint32_t addr) {
    float4 r;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w)
                 : "r"(addr));
    return r;
}
// m and v are touched once per call: no L1 allocation
__device__ __forceinline__ float4 ld_global_v4_stream(const float *p) {
    float4 r;
    asm volatile("ld.global.L1::no_allocate.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w)
                 : "l"(p));
    return r;
}
// read-only data that this SM reads once: no L1 allocation (the L1 left beside 200+ KB of
// shared memory is small and serves the epilogue)
__device__ __forceinline__ uint4 ld_global_nc_v4(const void *p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}
__device__ __forceinline__ void st_global_v4(float *p, float4 x) {
    asm volatile("st.global.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(x.x), "f"(x.y), "f"(x.z),
                 "f"(x.w)
                 : "memory");
}
// v += x as a reduction performed by the L2: the old value never enters the SM.  Every element
// is touched by exactly one thread per call, so the result is as deterministic as a store.
__device__ __forceinline__ void red_add_v4(float *p, float4 x) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(x.x), "f"(x.y), "f"(x.z),
                 "f"(x.w)
                 : "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, float x, float y, float z, float w) {
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(x), "f"(y), "f"(z),
                 "f"(w)
                 : "memory");
}

// Shared-memory matrix descriptor for an MN-major bf16 operand under the 128-byte
// swizzle.  Low word: start address >> 4 (bits 0..13) and leading byte offset >> 4
// (bits 16..29, the distance between 64-feature groups = one 8192-byte box).  High
// word: stride byte offset >> 4 (bits 32..45, the distance between 8-token groups =
// 1024 bytes), descriptor version 1 (bits 46..47), layout SWIZZLE_128B = 2 (bits 61..63).
// Only the start address changes between MMAs, so the issuing thread keeps the low word
// in a register and adds byte offsets >> 4 to it (no carry into bit 14: shared memory
// is smaller than 256 KB).
constexpr uint32_t kDescHi = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t addr) {
    return ((addr & 0x3ffffu) >> 4) | ((uint32_t)(BOX_BYTES >> 4) << 16);
}
__device__ __forceinline__ uint64_t smem_desc(uint32_t lo) {
    return ((uint64_t)kDescHi << 32) | (uint64_t)lo;
}

struct Barriers {
    uint64_t full[MAX_STAGES];
    uint64_t empty[MAX_STAGES];
    uint64_t acc_full[ACC_STAGES];
    uint64_t acc_empty[ACC_STAGES];
    uint64_t drain;
    // staged epilogue, per part buffer k and 32-row quarter q (one drain warp fills a quarter, two
    // streaming warps fold it): the quarter of buffer k holds its share of a part / is free again
    uint64_t g_full[2][4];
    uint64_t g_empty[2][4];
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(Barriers) <= SMEM_BAR_BYTES, "barrier block");

// The status block is global memory that the previous kernel of the stream (or the host's
// clearing of it) may still be writing under programmatic launch: the report waits for that
// kernel first (a no-op for roles that already have).
__device__ __forceinline__ void record_timeout(unsigned *status, Barriers *bars, unsigned site,
                                               unsigned tile) {
    *reinterpret_cast<volatile int *>(&bars->abort_flag) = 1;
    grid_dependency_wait();
    if (atomicCAS(status, (unsigned)kDevOk, (unsigned)kDevTimeout) == kDevOk) {
        status[1] = site;
        status[2] = tile;
    }
}

// Work list of a launch.  Items [0, split_from) are full tiles (TILE_M x 256), numbered
// with the index of the SHORTER tile dimension fastest: the ~74 tiles that run at the same
// time then span a nearly square block of the tile grid and share the fewest distinct operand
// blocks in the L2 (11008 x 4096 is 43 x 16 tiles: 74 consecutive tiles touch 5 row blocks and
// 16 column blocks with the column index fastest, 43 and 2 with the row index fastest).
// Calls of few tokens (the staged instance) are bound by the m, v traffic instead, and number
// the tiles with the column index fastest whatever the shape: the tiles in flight then cover
// whole rows of m and v (4096 x 4096, 2048 tokens: 74.0 us against 81.5; 1024 tokens: 62.9
// against 67.7; 4096 x 11008, 1024 tokens: 146.5 against 162.4).
// Items from split_from on are the two 128-column halves
// of the remaining full tiles: when the last round would occupy at most half of the CTA
// groups, halving its tiles halves its duration (the token sum of each half is still
// complete, so the square stays exact).
//
// One launch may cover several layers (adama_linear_wgrad_fold_multi): the work list is the
// layers' lists one after the other, and a CTA pair walks through it with a stride of the
// number of pairs.  The pairs that a layer's last round leaves idle therefore start on the
// next layer, the epilogue of a layer's last tile overlaps the next layer's first main loop,
// and set-up, pipeline fill and the one exposed epilogue are paid once per launch.
struct WorkItem {
    int m0, n0, width;
};
// Everything the kernel needs to know about one layer (kernel parameter space).
struct alignas(64) WgradLayer {
    CUtensorMap map_x, map_dy;             // 2-D views, one 64-feature x 64-token box per operation
    CUtensorMap map_x3, map_dy3, map_dy3h; // grouped 3-D views (d_in, d_out multiples of 64)
    float *m, *v;
    const __nv_bfloat16 *dy_raw;           // dY again, for the bias warps
    float *bias_m, *bias_v;                // null: the layer has no bias moments to fold
    long long ldmv, ldy;
    int tokens, d_in, d_out, grouped;
    int tiles_m, tiles_n;
    int split_from;   // layer-local item index from which items are 128-column halves
    int item_begin;   // index of the layer's first item in the launch's work list
    int col_fastest;  // tile numbering: column index fastest (else the row index)
};
constexpr int kMaxLayers = 8;
struct WgradTable {
    WgradLayer layer[kMaxLayers];
    int count;       // layers in this launch
    int num_items;   // work items of all layers
    int any_bias;    // some layer has bias moments: the CTAs carry the two bias warps
};
__device__ __forceinline__ WorkItem work_item(int w, int split_from, int tiles_m, int tiles_n,
                                              int col_fastest) {
    int full = w, half = 0, width = BN;
    if (w >= split_from) {
        const int j = w - split_from;
        full = split_from + (j >> 1);
        half = j & 1;
        width = BN / 2;
    }
    const int tm = col_fastest ? full / tiles_n : full % tiles_m;
    const int tn = col_fastest ? full % tiles_n : full / tiles_m;
    return {tm * Geo<>::TILE_M, tn * BN + half * (BN / 2), width};
}
// The layer that item `w` of the launch belongs to, and the item within that layer.
__device__ __forceinline__ const WgradLayer *layer_of(const WgradTable &tab, int w, WorkItem *wi) {
    int l = 0;
    while (l + 1 < tab.count && w >= tab.layer[l + 1].item_begin) ++l;
    const WgradLayer *L = &tab.layer[l];
    *wi = work_item(w - L->item_begin, L->split_from, L->tiles_m, L->tiles_n, L->col_fastest);
    return L;
}

template <bool STAGED>
__global__ void __launch_bounds__(STAGED ? STAGED_THREADS : MAX_THREADS, 1)
wgrad_fold_kernel(const __grid_constant__ WgradTable tab, float a, float b, unsigned *status,
                  unsigned long long wait_limit_ns, int withhold_last_load, int inputs_settled) {
    using G = Geo<STAGED>;
    constexpr int STAGES = G::STAGES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;  // swizzled tiles need 1024-B alignment
    uint8_t *smem = smem_raw + (base - raw_addr);
    Barriers *bars = reinterpret_cast<Barriers *>(smem + G::SMEM_BAR_OFF);
    volatile int *abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();  // position in the pair
    const int group = blockIdx.x / CTAS;                           // which pair
    const int num_groups = gridDim.x / CTAS;
    const int num_items = tab.num_items;
    // warps 2 .. 2+epi_warps-1: epilogue; with bias moments, BIAS_WARPS more after them
    // (staged: 4 drain warps take the epilogue's place, 8 streaming warps follow them)
    const int epi_warps = STAGED ? STAGED_DRAIN_WARPS
                                 : (int)blockDim.x / 32 - 2 - (tab.any_bias ? BIAS_WARPS : 0);
    const int first_bias_warp = 2 + epi_warps + (STAGED ? STAGED_STREAM_WARPS : 0);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&bars->full[s]), 1);
            mbar_init(smem_u32(&bars->empty[s]), 1);
        }
        for (int s = 0; s < ACC_STAGES; ++s) {
            mbar_init(smem_u32(&bars->acc_full[s]), 1);
            mbar_init(smem_u32(&bars->acc_empty[s]), epi_warps * CTAS);
        }
        mbar_init(smem_u32(&bars->drain), 1);
        for (int h = 0; h < 2; ++h) {
            for (int qq = 0; qq < 4; ++qq) {
                mbar_init(smem_u32(&bars->g_full[h][qq]), 1);
                mbar_init(smem_u32(&bars->g_empty[h][qq]), STAGED_STREAM_WARPS / STAGED_DRAIN_WARPS);
            }
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async_smem();
    }
    if (warp == 1) tmem_alloc(smem_u32(&bars->tmem_base));
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // the partner's barriers exist before anyone signals them
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(&bars->tmem_base);
    // Everything above touched only this CTA's shared and tensor memory, so it may run while
    // the previous kernel of the stream is still finishing; every role that reads or writes
    // global memory waits for that kernel first.  The next kernel may in turn set itself up
    // on SMs that this grid's CTAs leave early (the last round rarely fills all of them).
    grid_launch_dependents();

    if (warp == 0) {
        // ---------------- TMA producer (one thread of every CTA) ----------------
        if (lane == 0) {
            // X and dY may come from the kernel just before this one, unless the caller has
            // promised otherwise (ADAMA_INPUTS_SETTLED): then the first tiles' loads and MMAs run
            // beside that kernel's last round; m and v are still touched only after it
            if (!inputs_settled) grid_dependency_wait();
            int stage = 0;
            uint32_t phase = 0;
            uint32_t armed = 0;        // bit s: stage s has been armed at least once
            uint32_t last_parity = 0;  // bit s: parity of the phase last armed on stage s
            bool ok = true;
            const uint32_t full0 = smem_u32(&bars->full[0]);
            // the pair's loads are counted by the first CTA's barrier
            const uint32_t full0_lead = map_to_cta(full0, 0);
            for (int tile = group; tile < num_items && ok; tile += num_groups) {
                WorkItem wi;
                const WgradLayer *L = layer_of(tab, tile, &wi);
                const int num_kb = (L->tokens + BK - 1) / BK;
                const int cols_per_cta = wi.width / CTAS;  // dY columns this CTA stages
                const int b_boxes = cols_per_cta / GROUP;
                const int m0 = wi.m0 + (int)rank * G::ROWS_PER_CTA;
                const int n0 = wi.n0 + (int)rank * cols_per_cta;
                const uint32_t stage_tx =
                    (uint32_t)(G::A_STAGE_BYTES + b_boxes * BOX_BYTES) * CTAS;
                for (int kb = 0; kb < num_kb; ++kb) {
                    ok = mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1, abort_flag, wait_limit_ns);
                    if (!ok) {
                        record_timeout(status, bars, 1, (unsigned)tile);
                        break;
                    }
                    // Test hook (adama_debug_wgrad_expire_wait): the last stage of the launch's
                    // last work item is never loaded, so the issuer's wait for it must run out.
                    if (withhold_last_load && kb == num_kb - 1 && tile == num_items - 1) break;
                    const uint32_t bar = full0_lead + (uint32_t)stage * 8u;
                    const uint32_t sa = base + stage * G::STAGE_BYTES;
                    const uint32_t sb = sa + G::A_STAGE_BYTES;
                    // out-of-range parts of a box are zero-filled and still counted
                    if (rank == 0) mbar_arrive_expect_tx(full0 + (uint32_t)stage * 8u, stage_tx);
                    if (L->grouped) {
                        // d_in, d_out multiples of 64: one operation per operand
                        tma_load_3d(sa, &L->map_x3, kb * BK, m0 / GROUP, bar);
                        tma_load_3d(sb, b_boxes == G::B_BOXES ? &L->map_dy3 : &L->map_dy3h, kb * BK,
                                          n0 / GROUP, bar);
                    } else {
#pragma unroll
                        for (int j = 0; j < G::A_BOXES; ++j)
                            tma_load_2d(sa + j * BOX_BYTES, &L->map_x, m0 + j * GROUP, kb * BK,
                                              bar);
                        for (int j = 0; j < b_boxes; ++j)
                            tma_load_2d(sb + j * BOX_BYTES, &L->map_dy, n0 + j * GROUP, kb * BK,
                                              bar);
                    }
                    armed |= 1u << stage;
                    last_parity = (last_parity & ~(1u << stage)) | (phase << stage);
                    if (++stage == STAGES) {
                        stage = 0;
                        phase ^= 1;
                    }
                }
            }
            if (*abort_flag && rank == 0) {
                // leave no copy in flight behind: wait (bounded) for every armed stage to land
                int never = 0;
                for (int s = 0; s < STAGES; ++s)
                    if (armed & (1u << s))
                        mbar_wait(full0 + (uint32_t)s * 8u, (last_parity >> s) & 1u, &never,
                                  kDrainLimitNs);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer (one thread of the pair's first CTA) ----------------
        // The tensor core runs in step with the issuing thread (few MMAs can be queued), so
        // whatever the thread does between two MMAs is exposed.  The barrier of the NEXT
        // stage is therefore probed while the current stage's MMAs are still executing.
        if (rank == 0 && lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int it = 0;
            const uint32_t desc_lo0 = smem_desc_lo(base);  // operand A of stage 0
            const uint32_t full0 = smem_u32(&bars->full[0]);
            uint32_t empty_bar0[CTAS];  // empty[0] in each CTA of the pair
#pragma unroll
            for (int r = 0; r < CTAS; ++r)
                empty_bar0[r] = map_to_cta(smem_u32(&bars->empty[0]), r);
            bool next_ready = false;  // full[stage] already seen complete by a probe
            for (int tile = group; tile < num_items && ok; tile += num_groups, ++it) {
                const int as = it & 1;
                const uint32_t aphase = (uint32_t)(it >> 1) & 1u;
                WorkItem wi;
                const WgradLayer *L = layer_of(tab, tile, &wi);
                const int num_kb = (L->tokens + BK - 1) / BK;
                const uint32_t idesc = G::INSTR_DESC_NO_N | ((uint32_t)(wi.width >> 3) << 17);
                ok = mbar_wait(smem_u32(&bars->acc_empty[as]), aphase ^ 1, abort_flag, wait_limit_ns);
                if (!ok) {
                    record_timeout(status, bars, 2, (unsigned)tile);
                    break;
                }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(as * BN);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!next_ready) {
                        ok = mbar_wait(full0 + (uint32_t)stage * 8u, phase, abort_flag, wait_limit_ns);
                        if (!ok) {
                            record_timeout(status, bars, 3, (unsigned)tile);
                            break;
                        }
                    }
                    tc_fence_after();
                    const uint32_t a_lo = desc_lo0 + (uint32_t)stage * (G::STAGE_BYTES >> 4);
                    const uint32_t b_lo = a_lo + (G::A_STAGE_BYTES >> 4);
                    int nstage = stage + 1;
                    uint32_t nphase = phase;
                    if (nstage == STAGES) {
                        nstage = 0;
                        nphase ^= 1;
                    }
                    // 16 tokens further = 16 rows of 128 bytes
                    constexpr uint32_t kstep = (UMMA_K * 128) >> 4;
                    constexpr int KSTEPS = BK / UMMA_K;
#pragma unroll
                    for (int k = 0; k < KSTEPS - 1; ++k)
                        tc_mma(tmem_d, smem_desc(a_lo + k * kstep),
                                     smem_desc(b_lo + k * kstep), idesc, (kb | k) != 0 ? 1u : 0u);
                    // look ahead while those execute (a stale "ready" cannot occur: the
                    // barrier cannot advance two phases before this thread frees the stage)
                    next_ready = mbar_try_wait(full0 + (uint32_t)nstage * 8u, nphase);
                    tc_mma(tmem_d, smem_desc(a_lo + (KSTEPS - 1) * kstep),
                                 smem_desc(b_lo + (KSTEPS - 1) * kstep), idesc, 1u);
                    // the stage is free, in every CTA of the pair, once these MMAs retire
#pragma unroll
                    for (int r = 0; r < CTAS; ++r)
                        tc_commit(empty_bar0[r] + (uint32_t)stage * 8u);
                    stage = nstage;
                    phase = nphase;
                }
                if (ok) {
                    const uint32_t f = smem_u32(&bars->acc_full[as]);
#pragma unroll
                    for (int r = 0; r < CTAS; ++r) tc_commit(map_to_cta(f, r));
                }
            }
            if (*abort_flag) {
                // let issued MMAs retire before TMEM is given back
                tc_commit(smem_u32(&bars->drain));
                int never = 0;
                mbar_wait(smem_u32(&bars->drain), 0, &never, kDrainLimitNs);
            }
        }
        __syncwarp();
    } else if (STAGED && warp >= 2 + STAGED_DRAIN_WARPS && warp < 2 + STAGED_DRAIN_WARPS + STAGED_STREAM_WARPS) {
        // ---------------- staged epilogue, streaming side: shared-memory tile -> m, v ----------------
        // A warp owns 16 rows of the CTA's 128; the tile comes in parts of PART_COLS columns, so
        // that one part is folded while the drain warps copy the next.  A warp instruction covers
        // 32/LPR rows x PART_COLS*4 contiguous bytes.  m is read, folded and written back; v takes
        // its increment through an L2 reduction, so only half of the state traffic enters the SM.
        // The eight m loads of the NEXT part (or of the next tile's first part) are issued before
        // the current part is folded: the loads never drain between parts.  Buffers change hands per
        // 32-row quarter (drain warp q <-> streaming warps 2q, 2q+1), not per part: with one barrier
        // for all twelve warps the slowest warp of either side gated every hand-over and copy and
        // fold ran one after the other (4.4 us per part at 256 tokens).
        const int sw_id = warp - (2 + STAGED_DRAIN_WARPS);
        const uint32_t gbuf = base + G::SMEM_EPI_OFF;
        constexpr int LPR = PART_COLS / 4;   // lanes per row: a warp instruction covers 32 / LPR rows
        constexpr int RPI = 32 / LPR;
        constexpr int PITCH = PART_COLS * 4;  // bytes per row of a part buffer
        static_assert(8 * RPI == 16, "a warp's 16 rows of a part are one batch of eight loads");
        const int sub = lane / LPR, cl = lane % LPR;
        const int lrow0 = sw_id * 16 + sub;  // this thread's first row of the CTA's 128
        bool ok = true;
        uint32_t use_bits = 0;    // bit k: parity of how often part buffer k has been used
        grid_dependency_wait();   // m and v may still be written by the previous call

        struct Part {
            float *pm, *pv;
            long long ldmv;
            int row_first, gcol, d_in, d_out;
            bool col_vec;
        };
        auto part_at = [&](int tile, int part_i) {
            WorkItem wi;
            const WgradLayer *L = layer_of(tab, tile, &wi);
            Part u;
            u.ldmv = L->ldmv;
            u.d_in = L->d_in;
            u.d_out = L->d_out;
            u.row_first = wi.m0 + (int)rank * G::ROWS_PER_CTA + lrow0;
            u.gcol = wi.n0 + part_i * PART_COLS + cl * 4;
            u.col_vec = u.gcol + 4 <= u.d_out;  // whole group of four columns inside
            u.pm = L->m + (long long)u.row_first * u.ldmv + u.gcol;
            u.pv = L->v + (long long)u.row_first * u.ldmv + u.gcol;
            return u;
        };
        auto load_m = [&](const Part &u, float4(&mm)[8]) {
            if (u.col_vec) {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (u.row_first + i * RPI < u.d_in)
                        mm[i] = ld_global_v4_stream(u.pm + (long long)(i * RPI) * u.ldmv);
            }
        };
        // waits for part buffer k to hold the part, folds it, hands the buffer back
        auto fold_part = [&](const Part &u, float4(&mm)[8], int k, int tile) {
            ok = mbar_wait(smem_u32(&bars->g_full[k][sw_id >> 1]), (use_bits >> k) & 1u, abort_flag, wait_limit_ns);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) {
                if (lane == 0) record_timeout(status, bars, 7, (unsigned)tile);
                return;
            }
            use_bits ^= 1u << k;
            const uint32_t pbuf = gbuf + (uint32_t)k * PART_BYTES;
            if (u.col_vec) {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (u.row_first + i * RPI < u.d_in) {
                        const int lrow = lrow0 + i * RPI;
                        const float4 g = ld_shared_v4(pbuf + (uint32_t)lrow * PITCH +
                                                      (uint32_t)((cl ^ (lrow & 7)) << 4));
                        float4 &x = mm[i];
                        x.x = fmaf(a, g.x, x.x);
                        x.y = fmaf(a, g.y, x.y);
                        x.z = fmaf(a, g.z, x.z);
                        x.w = fmaf(a, g.w, x.w);
                        st_global_v4(u.pm + (long long)(i * RPI) * u.ldmv, x);
                        red_add_v4(u.pv + (long long)(i * RPI) * u.ldmv,
                                   make_float4((b * g.x) * g.x, (b * g.y) * g.y, (b * g.z) * g.z,
                                               (b * g.w) * g.w));
                    }
            } else if (u.gcol < u.d_out) {
                // last, partial group of four columns: element-wise
                for (int i = 0; i < 8; ++i) {
                    const int lrow = lrow0 + i * RPI;
                    if (u.row_first + i * RPI >= u.d_in) break;
                    const float4 g = ld_shared_v4(pbuf + (uint32_t)lrow * PITCH +
                                                  (uint32_t)((cl ^ (lrow & 7)) << 4));
                    const float ge[4] = {g.x, g.y, g.z, g.w};
                    for (int e = 0; e < 4; ++e)
                        if (u.gcol + e < u.d_out) {
                            float *qm = u.pm + (long long)(i * RPI) * u.ldmv + e;
                            float *qv = u.pv + (long long)(i * RPI) * u.ldmv + e;
                            *qm = fmaf(a, ge[e], *qm);
                            *qv = __fadd_rn(*qv, __fmul_rn(__fmul_rn(b, ge[e]), ge[e]));  // as the reduction rounds
                        }
                }
            }
            __syncwarp();  // every lane has read its share of this part
            if (lane == 0) mbar_arrive(smem_u32(&bars->g_empty[k][sw_id >> 1]));
        };

        if (group < num_items) {
            float4 m_a[8], m_b[8];
            Part u_a = part_at(group, 0), u_b = u_a;
            load_m(u_a, m_a);
            for (int tile = group; tile < num_items && ok; tile += num_groups) {
                // parts per tile: 4 (full tile) or 2 (half tile); part i lives in buffer i & 1
                WorkItem wi_t;
                layer_of(tab, tile, &wi_t);
                const int nparts = wi_t.width / PART_COLS;
                for (int part_i = 0; part_i < nparts && ok; part_i += 2) {
                    u_b = part_at(tile, part_i + 1);
                    load_m(u_b, m_b);
                    fold_part(u_a, m_a, 0, tile);
                    if (!ok) break;
                    if (part_i + 2 < nparts) {
                        u_a = part_at(tile, part_i + 2);
                        load_m(u_a, m_a);
                    } else if (tile + num_groups < num_items) {
                        u_a = part_at(tile + num_groups, 0);
                        load_m(u_a, m_a);
                    }
                    fold_part(u_b, m_b, 1, tile);
                }
            }
        }
    } else if (warp >= first_bias_warp) {
        // ---------------- bias gradient: column sums of dY, folded into the bias moments ----------------
        // Two extra warps (present only when bias moments were passed) work through the layer's
        // bias gradient while the other roles run the tiles, straight from global memory (the
        // producer pulls the same dY through the L2 anyway).  A CTA takes whole 32-column slabs
        // over ALL tokens, so a token sum is complete before it is squared and no CTA depends
        // on another: a warp load covers 8 rows x 64 bytes, 8 loads in flight per thread (4 make these
        // warps the last to finish on wide layers, 16 take more from the main loop's loads), sums
        // combined across the 8 row lanes by shuffles and across the two warps through shared
        // memory, in fixed order.  These warps wait on no mbarrier, so the named barrier
        // between them cannot be left waiting by a role that gave up.
        grid_dependency_wait();
        const int ew = warp - first_bias_warp;
        float *red = reinterpret_cast<float *>(smem + G::SMEM_BIAS_OFF);  // [BIAS_WARPS][32]
        const int rsub = lane >> 2;  // row within a group of 8
        const int cq = lane & 3;     // 16-byte chunk of the slab's 64-byte row segment
        const int step = BIAS_WARPS * 8;
        for (int l = 0; l < tab.count; ++l) {
        const WgradLayer *L = &tab.layer[l];
        float *bias_m = L->bias_m, *bias_v = L->bias_v;
        if (bias_m == nullptr) continue;  // (uniform over the two warps)
        const int d_out = L->d_out, tokens = L->tokens;
        const long long ldy = L->ldy;
        const __nv_bfloat16 *dy_raw = L->dy_raw;
        const int slabs = (d_out + 31) / 32;
        for (int slab = (int)blockIdx.x; slab < slabs; slab += (int)gridDim.x) {
            const int col = slab * 32 + cq * 8;
            float acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = 0.f;
            if (col + 8 <= d_out) {
                const __nv_bfloat16 *src = dy_raw + col;
                int tau = ew * 8 + rsub;
                for (; tau + (BIAS_UNROLL - 1) * step < tokens; tau += BIAS_UNROLL * step) {
                    uint4 x[BIAS_UNROLL];
#pragma unroll
                    for (int u = 0; u < BIAS_UNROLL; ++u)
                        x[u] = ld_global_nc_v4(src + (long long)(tau + u * step) * ldy);
#pragma unroll
                    for (int u = 0; u < BIAS_UNROLL; ++u) {
                        const unsigned wds[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            acc[2 * k] += __uint_as_float(wds[k] << 16);
                            acc[2 * k + 1] += __uint_as_float(wds[k] & 0xffff0000u);
                        }
                    }
                }
                for (; tau < tokens; tau += step) {
                    const uint4 x = ld_global_nc_v4(src + (long long)tau * ldy);
                    const unsigned wds[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        acc[2 * k] += __uint_as_float(wds[k] << 16);
                        acc[2 * k + 1] += __uint_as_float(wds[k] & 0xffff0000u);
                    }
                }
            } else {
                // ragged last columns: element-wise, bounds-checked
                for (int tau = ew * 8 + rsub; tau < tokens; tau += step)
                    for (int e = 0; e < 8; ++e)
                        if (col + e < d_out)
                            acc[e] += __bfloat162float(dy_raw[(long long)tau * ldy + col + e]);
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], 4);
                acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], 8);
                acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], 16);
            }
            if (rsub == 0) {
#pragma unroll
                for (int e = 0; e < 8; ++e) red[ew * 32 + cq * 8 + e] = acc[e];
            }
            asm volatile("bar.sync 1, %0;" ::"r"(BIAS_WARPS * 32) : "memory");
            if (ew == 0) {
                const int qcol = slab * 32 + lane;
                if (qcol < d_out) {
                    float g = 0.f;
#pragma unroll
                    for (int w2 = 0; w2 < BIAS_WARPS; ++w2) g += red[w2 * 32 + lane];
                    bias_m[qcol] = fmaf(a, g, bias_m[qcol]);
                    bias_v[qcol] = fmaf(b * g, g, bias_v[qcol]);
                }
            }
            asm volatile("bar.sync 1, %0;" ::"r"(BIAS_WARPS * 32) : "memory");
        }
        }  // layers
    } else {
        if constexpr (STAGED) {
            // ---------------- staged epilogue, drain side: accumulator -> shared-memory tile ----------------
            // Thread = accumulator row; 16-byte chunk j of row r sits at chunk (j ^ (r & 7)), so these
            // row-per-thread writes and the streaming warps' row-contiguous reads are conflict-free.
            const int q = warp & 3;
            const uint32_t gbuf = base + G::SMEM_EPI_OFF;
            const int lrow = q * EPI_ROWS + lane;
            bool ok = true;
            int it = 0;
            uint32_t use_bits = 0;  // bit k: parity of how often part buffer k has been filled
            for (int tile = group; tile < num_items && ok; tile += num_groups, ++it) {
                const int as = it & 1;
                const uint32_t aphase = (uint32_t)(it >> 1) & 1u;
                WorkItem wi;
                layer_of(tab, tile, &wi);
                ok = mbar_wait(smem_u32(&bars->acc_full[as]), aphase, abort_flag, wait_limit_ns);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) {
                    if (lane == 0) record_timeout(status, bars, 4, (unsigned)tile);
                    break;
                }
                tc_fence_after();
                const uint32_t taddr0 =
                    tmem_base + ((uint32_t)(q * EPI_ROWS) << 16) + (uint32_t)(as * BN);
                for (int part_i = 0; part_i < wi.width / PART_COLS; ++part_i) {
                    if (!ok) continue;
                    const int k = part_i & 1;
                    // the streaming warps must be done with this buffer's previous contents
                    ok = mbar_wait(smem_u32(&bars->g_empty[k][q]), ((use_bits >> k) & 1u) ^ 1u, abort_flag, wait_limit_ns);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) {
                        if (lane == 0) record_timeout(status, bars, 6, (unsigned)tile);
                        continue;
                    }
                    use_bits ^= 1u << k;
                    const uint32_t pbuf = gbuf + (uint32_t)k * PART_BYTES;
                    constexpr int CPP = PART_COLS / EPI_COLS;  // 32-column chunks per part
                    for (int c = 0; c < CPP; ++c) {
                        uint32_t r[32];
                        tc_ld_32x32(taddr0 + (uint32_t)((part_i * CPP + c) * EPI_COLS), r);
                        tc_wait_ld();
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            st_shared_v4(pbuf + (uint32_t)lrow * (PART_COLS * 4) +
                                             (uint32_t)(((c * 8 + j) ^ (lrow & 7)) << 4),
                                         __uint_as_float(r[4 * j + 0]), __uint_as_float(r[4 * j + 1]),
                                         __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars->g_full[k][q]));
                }
                if (!ok) break;
                // the accumulator stage may be overwritten
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    const uint32_t e = smem_u32(&bars->acc_empty[as]);
                    mbar_arrive_cluster(map_to_cta(e, 0));
                }
            }
        } else {
        // ---------------- epilogue: m = fma(a, G, m), v += (b*G)*G ----------------
        // m is read, folded and written back by the SM; v takes its increment through an L2
        // reduction (red.global.add), so that only half of the state traffic enters the SM:
        // the SM's inbound port, which also carries the operand tiles, is what bounds the
        // main loop that this epilogue overlaps.  The m loads of a tile's first chunk are issued
        // before the wait for its accumulator.
        const int q = warp & 3;            // TMEM lane quarter this warp may read
        const int part = (warp - 2) >> 2;  // which part of the tile's columns it handles
        const int col_split = epi_warps / 4;  // 1 or 2 warps per lane quarter
        const uint32_t sm_g = base + G::SMEM_EPI_OFF + (uint32_t)(warp - 2) * EPI_BUF_BYTES;
        // staging buffer: 32 rows of 128 bytes; 16-byte chunk j of row r sits at (j ^ (r & 7)),
        // which makes both the row-per-thread writes and the row-segment reads conflict-free
        const uint32_t row_off = (uint32_t)lane * 128u;
        const uint32_t sw = (uint32_t)(lane & 7);
        // coalesced side: a quarter-warp covers 128 contiguous bytes of one row
        const int sub_row = lane >> 3;  // 0..3
        const int c4 = lane & 7;        // which float4 of the 32-column chunk
        bool ok = true;
        int it = 0;
        grid_dependency_wait();  // m and v may still be written by the previous call

        // one 32 x 32 chunk of the tile: geometry, m loads, fold
        struct Chunk {
            long long off0;
            int col0;
            bool inside, interior;
        };
        // the layer of the tile at hand (set per tile; the helpers below read it)
        float *m_out = nullptr, *v_out = nullptr;
        long long ldmv = 0;
        int d_in = 0, d_out = 0;
        auto chunk_at = [&](const WorkItem &wi, int row0, int c) {
            Chunk ch;
            ch.col0 = wi.n0 + c * EPI_COLS;
            ch.inside = row0 < d_in && ch.col0 < d_out;
            ch.interior = row0 + EPI_ROWS <= d_in && ch.col0 + EPI_COLS <= d_out;
            ch.off0 = (long long)(row0 + sub_row) * ldmv + ch.col0 + c4 * 4;
            return ch;
        };
        auto load_m = [&](const Chunk &ch, float4(&mm)[8]) {
            if (ch.interior) {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    mm[i] = ld_global_v4_stream(m_out + ch.off0 + (long long)i * 4 * ldmv);
            }
        };
        auto fold_chunk = [&](const Chunk &ch, float4(&mm)[8], uint32_t taddr, int row0) {
            if (!ch.inside) return;  // chunks wholly outside the matrix are skipped
            uint32_t r[32];
            tc_ld_32x32(taddr, r);
            tc_wait_ld();
            __syncwarp();  // the previous chunk has been read out of the buffer
#pragma unroll
            for (int j = 0; j < 8; ++j)
                st_shared_v4(sm_g + row_off + ((((uint32_t)j) ^ sw) << 4),
                             __uint_as_float(r[4 * j + 0]), __uint_as_float(r[4 * j + 1]),
                             __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
            __syncwarp();
            if (ch.interior) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int row = i * 4 + sub_row;
                    const float4 g = ld_shared_v4(sm_g + (uint32_t)row * 128u +
                                                  (uint32_t)((c4 ^ (row & 7)) << 4));
                    mm[i].x = fmaf(a, g.x, mm[i].x);
                    mm[i].y = fmaf(a, g.y, mm[i].y);
                    mm[i].z = fmaf(a, g.z, mm[i].z);
                    mm[i].w = fmaf(a, g.w, mm[i].w);
                    st_global_v4(m_out + ch.off0 + (long long)i * 4 * ldmv, mm[i]);
                    red_add_v4(v_out + ch.off0 + (long long)i * 4 * ldmv,
                               make_float4((b * g.x) * g.x, (b * g.y) * g.y, (b * g.z) * g.z,
                                           (b * g.w) * g.w));
                }
            } else {
                // ragged edge of the matrix: element-wise, bounds-checked
                for (int i = 0; i < 8; ++i) {
                    const int row = i * 4 + sub_row;
                    if (row0 + row >= d_in) continue;
                    const float4 g = ld_shared_v4(sm_g + (uint32_t)row * 128u +
                                                  (uint32_t)((c4 ^ (row & 7)) << 4));
                    const float ge[4] = {g.x, g.y, g.z, g.w};
                    float *pm = m_out + ch.off0 + (long long)i * 4 * ldmv;
                    float *pv = v_out + ch.off0 + (long long)i * 4 * ldmv;
                    for (int e = 0; e < 4; ++e)
                        if (ch.col0 + c4 * 4 + e < d_out) {
                            pm[e] = fmaf(a, ge[e], pm[e]);
                            pv[e] = __fadd_rn(pv[e], __fmul_rn(__fmul_rn(b, ge[e]), ge[e]));  // as the reduction rounds
                        }
                }
            }
        };

        for (int tile = group; tile < num_items && ok; tile += num_groups, ++it) {
            const int as = it & 1;
            const uint32_t aphase = (uint32_t)(it >> 1) & 1u;
            WorkItem wi;
            const WgradLayer *L = layer_of(tab, tile, &wi);
            m_out = L->m;
            v_out = L->v;
            ldmv = L->ldmv;
            d_in = L->d_in;
            d_out = L->d_out;
            const int row0 = wi.m0 + (int)rank * G::ROWS_PER_CTA + q * EPI_ROWS;
            const int chunks = wi.width / (col_split * EPI_COLS);  // chunks per warp
            const int c_first = part * chunks;
            float4 mm[8];
            Chunk ch = chunk_at(wi, row0, c_first);
            load_m(ch, mm);  // in flight while the tile's main loop still runs
            ok = mbar_wait(smem_u32(&bars->acc_full[as]), aphase, abort_flag, wait_limit_ns);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) {
                if (lane == 0) record_timeout(status, bars, 4, (unsigned)tile);
                break;
            }
            tc_fence_after();
            const uint32_t taddr0 =
                tmem_base + ((uint32_t)(q * EPI_ROWS) << 16) + (uint32_t)(as * BN);
            for (int cc = 0; cc < chunks; ++cc) {
                if (cc > 0) {
                    ch = chunk_at(wi, row0, c_first + cc);
                    load_m(ch, mm);
                }
                fold_chunk(ch, mm, taddr0 + (uint32_t)((c_first + cc) * EPI_COLS), row0);
            }
            // accumulator stage may now be overwritten by the pair's MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                const uint32_t e = smem_u32(&bars->acc_empty[as]);
                mbar_arrive_cluster(map_to_cta(e, 0));
            }
        }
        }  // !STAGED
    }

    tc_fence_before();
    __syncthreads();
    // neither CTA of a pair may retire while the other can still read its shared memory
    // or signal its barriers
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base);
    }
}

// ---- host side -----------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
// One-time set-up, guarded by g_setup_mutex: the driver's tensor-map encoder once per process,
// the kernels' shared-memory limit once per DEVICE (cudaFuncSetAttribute applies to the
// current device only).
std::mutex g_setup_mutex;
constexpr int kMaxTrackedDevices = 64;
bool g_attr_set[kMaxTrackedDevices] = {};

// 2-D row-major tensor [rows, cols] with row pitch `ld` elements, box [box_rows, box_cols].
bool encode_2d(CUtensorMap *map, CUtensorMapDataType dt, size_t elem, const void *ptr,
               uint64_t cols, uint64_t rows, uint64_t ld, uint32_t box_cols, uint32_t box_rows,
               CUtensorMapL2promotion promo) {
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld * elem};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(map, dt, 2, const_cast<void *>(ptr), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, promo,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// 3-D view of a row-major [tokens, d] bf16 matrix with d a multiple of 64:
// {64 features (contiguous), tokens (pitch ld), d/64 groups (128 bytes apart)}; a box takes
// 64 features x box_tokens x box_groups and lands group after group, 8192 bytes each.
bool encode_grouped(CUtensorMap *map, const void *ptr, uint64_t d, uint64_t tokens, uint64_t ld,
                    uint32_t box_tokens, uint32_t box_groups) {
    cuuint64_t dims[3] = {GROUP, tokens, d / GROUP};
    cuuint64_t strides[2] = {ld * 2, GROUP * 2};
    cuuint32_t box[3] = {GROUP, box_tokens, box_groups};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims,
                          strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

}  // namespace

cudaError_t wgrad_fold_setup(const char **msg) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000,
                                                         cudaEnableDefault, &qres);
        if (e != cudaSuccess) {
            *msg = "cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)";
            return e;
        }
        if (qres != cudaDriverEntryPointSuccess || !fn) {
            *msg = "driver has no cuTensorMapEncodeTiled";
            return cudaErrorNotSupported;
        }
        g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    return cudaSuccess;
}

static bool attr_needed(int device) {
    return device < 0 || device >= kMaxTrackedDevices || !g_attr_set[device];
}

int wgrad_setup_state(int device) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    return (g_encode ? 1 : 0) | (attr_needed(device) ? 0 : 2);
}

// The kernels' dynamic shared-memory limit on the CURRENT device (set once per device).
static cudaError_t ensure_device_attributes(const char **msg) {
    int device = -1;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) {
        *msg = "cudaGetDevice";
        return e;
    }
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!attr_needed(device)) return cudaSuccess;
    e = cudaFuncSetAttribute(wgrad_fold_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Geo<false>::SMEM_BYTES);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(wgrad_fold_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 Geo<true>::SMEM_BYTES);
    if (e != cudaSuccess) {
        *msg = "cudaFuncSetAttribute(wgrad_fold_kernel)";
        return e;
    }
    // devices beyond the table are simply set up on every call
    if (device >= 0 && device < kMaxTrackedDevices) g_attr_set[device] = true;
    return cudaSuccess;
}

// Fills one layer's entry of the kernel's table; *tiles = the layer's full 256x256 tiles.
static bool fill_layer(const WgradArgs &p, WgradLayer *L, int *tiles) {
    bool ok = encode_2d(&L->map_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p.X, (uint64_t)p.d_in,
                        (uint64_t)p.tokens, (uint64_t)p.ldx, GROUP, BK,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B) &&
              encode_2d(&L->map_dy, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p.dY, (uint64_t)p.d_out,
                        (uint64_t)p.tokens, (uint64_t)p.ldy, GROUP, BK,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
    // grouped loads need whole 64-feature groups in both operands
    L->map_x3 = L->map_x;
    L->map_dy3 = L->map_dy;
    L->map_dy3h = L->map_dy;
    L->grouped = (p.d_in % GROUP == 0 && p.d_out % GROUP == 0 && !p.variant.box_loads) ? 1 : 0;
    if (ok && L->grouped)
        ok = encode_grouped(&L->map_x3, p.X, (uint64_t)p.d_in, (uint64_t)p.tokens, (uint64_t)p.ldx,
                            BK, Geo<>::A_BOXES) &&
             encode_grouped(&L->map_dy3, p.dY, (uint64_t)p.d_out, (uint64_t)p.tokens,
                            (uint64_t)p.ldy, BK, Geo<>::B_BOXES) &&
             encode_grouped(&L->map_dy3h, p.dY, (uint64_t)p.d_out, (uint64_t)p.tokens,
                            (uint64_t)p.ldy, BK, Geo<>::B_BOXES / 2);
    L->m = p.m;
    L->v = p.v;
    L->dy_raw = static_cast<const __nv_bfloat16 *>(p.dY);
    L->bias_m = p.bias_m;
    L->bias_v = p.bias_v;
    L->ldmv = (long long)p.ldmv;
    L->ldy = (long long)p.ldy;
    L->tokens = p.tokens;
    L->d_in = p.d_in;
    L->d_out = p.d_out;
    L->tiles_m = (p.d_in + Geo<>::TILE_M - 1) / Geo<>::TILE_M;
    L->tiles_n = (p.d_out + BN - 1) / BN;
    *tiles = L->tiles_m * L->tiles_n;
    L->split_from = *tiles;  // no halves unless the launch's tail says so
    L->col_fastest = L->tiles_n < L->tiles_m ? 1 : 0;  // shorter dimension fastest (see WorkItem)
    return ok;
}

cudaError_t launch_wgrad_fold_multi(const WgradArgs *layers, int count, const char **msg) {
    if (count < 1 || count > kMaxWgradLayers) {
        *msg = "wgrad_fold: layer count out of range";
        return cudaErrorInvalidValue;
    }
    cudaError_t e = wgrad_fold_setup(msg);
    if (e == cudaSuccess) e = ensure_device_attributes(msg);
    if (e != cudaSuccess) return e;
    const WgradArgs &p = layers[0];  // stream, status block, constants, variant: the launch's
    static_assert(kMaxWgradLayers == kMaxLayers, "table size");
    WgradTable tab = {};
    tab.count = count;
    int items = 0, max_tokens = 0, min_tokens = layers[0].tokens;
    int tiles_of[kMaxLayers];
    for (int l = 0; l < count; ++l) {
        if (!fill_layer(layers[l], &tab.layer[l], &tiles_of[l])) {
            *msg = "cuTensorMapEncodeTiled rejected a tensor";
            return cudaErrorInvalidValue;
        }
        tab.layer[l].item_begin = items;
        items += tiles_of[l];
        if (layers[l].bias_m) tab.any_bias = 1;
        max_tokens = layers[l].tokens > max_tokens ? layers[l].tokens : max_tokens;
        min_tokens = layers[l].tokens < min_tokens ? layers[l].tokens : min_tokens;
    }
    *msg = "wgrad_fold launch";
    const int max_groups = p.sm_count / 2;
    // Tail balancing: if the launch's last round would keep at most half of the groups busy, its
    // tiles (the last layer's last ones) are issued as 128-column halves (see WorkItem).
    const int rest = items % max_groups;
    if (rest > 0 && 2 * rest <= max_groups && rest <= tiles_of[count - 1]) {
        tab.layer[count - 1].split_from = tiles_of[count - 1] - rest;
        items += rest;
    }
    tab.num_items = items;
    const int groups = items < max_groups ? items : max_groups;
    // 8 epilogue warps when no CTA group gets a second tile (exposed epilogue) or when the
    // contraction is short (up to 2048 tokens the m, v traffic of the epilogue, not the tensor
    // cores, bounds the call: 4096x4096 with 1024 tokens 78.9 vs 82.9 us), else 4
    const bool wide = p.variant.epi_warps ? p.variant.epi_warps == 8
                                          : (items <= max_groups || max_tokens <= 2048);
    const int threads = 32 * (2 + (wide ? MAX_EPI_WARPS : 4) + (tab.any_bias ? BIAS_WARPS : 0));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * groups), 1, 1);
    cfg.blockDim = dim3((unsigned)threads, 1, 1);
    // calls of few tokens: staged epilogue (see STAGED_RING)
    // (4096x4096, L2 flushed, staged vs direct epilogue, us: 256 tokens 65.6 vs 75.8, 1024: 69.7 vs
    // 79.9, 2048: 75.8 vs 82.0, 3072: 94.2 vs 92.2, 4096: 114.7 vs 110.6.  With 128-column parts and
    // the 3-stage ring they leave: 66.6, 71.7, 92.2 at 256, 1024, 2048 tokens.)
    const bool staged = p.variant.epilogue ? p.variant.epilogue == 2 : max_tokens <= 2048;
    cfg.dynamicSmemBytes = staged ? Geo<true>::SMEM_BYTES : Geo<>::SMEM_BYTES;
    if (staged)
        for (int l = 0; l < count; ++l) tab.layer[l].col_fastest = 1;  // whole rows of m, v in flight
    if (staged) cfg.blockDim = dim3((unsigned)(STAGED_THREADS - (tab.any_bias ? 0 : 32 * BIAS_WARPS)), 1, 1);
    cfg.stream = p.stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // programmatic launch: this kernel's set-up may overlap the tail of the kernel before it
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.variant.no_pdl ? 1 : 2;
    const unsigned long long limit = p.wait_limit_ns ? p.wait_limit_ns : kDefaultWaitLimitNs;
    return cudaLaunchKernelEx(&cfg, staged ? wgrad_fold_kernel<true> : wgrad_fold_kernel<false>, tab,
                              p.c.a, p.c.b, p.status, limit, p.withhold_last_load, p.inputs_settled);
}

cudaError_t launch_wgrad_fold(const WgradArgs &p, const char **msg) {
    return launch_wgrad_fold_multi(&p, 1, msg);
}

}  // namespace adama

// ---- allocation-free entry point ------------------------------------------------------------
//
// The fused kernel needs one piece of global memory besides its inputs and outputs: the
// 256-byte status block in which a CTA records that a bounded wait ran out.  A context
// gets that block from cudaMalloc.  Code that must not allocate -- a training loop whose
// device memory belongs entirely to a framework's pool, a plug-in called while another
// component holds the allocator lock, a caller past its memory budget -- cannot create a
// context, so this entry point needs none: the block lives in the library image itself.

namespace adama {
namespace {

constexpr size_t kStaticScratchBytes = 256;  // the whole need of the kernel, whatever the shapes
constexpr int kMaxDevices = 64;

// One copy per GPU that loads the library, held until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

struct StaticSetup {
    unsigned *scratch = nullptr;  // DEVICE address of g_static_scratch on that GPU
    int sm_count = 0;
};
StaticSetup g_static_setup[kMaxDevices];
std::mutex g_static_mutex;  // the table is filled in by whichever thread calls first

// In host code `g_static_scratch` is only a handle for the runtime, not an address a kernel
// can use; the device address has to be asked for, with the right device current.
cudaError_t static_setup_for_current_device(int device, StaticSetup **out, const char **msg) {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticSetup &s = g_static_setup[device];
    if (!s.scratch) {
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) {
            *msg = "cudaGetSymbolAddress(static scratch)";
            return e;
        }
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
        if (e != cudaSuccess) {
            *msg = "cudaDeviceGetAttribute(multiProcessorCount)";
            return e;
        }
        s.sm_count = sms;
        s.scratch = static_cast<unsigned *>(ptr);
    }
    *out = &s;
    return cudaSuccess;
}

void set_msg(char *err, size_t err_len, const char *text, const char *detail = nullptr) {
    if (!err || err_len == 0) return;
    size_t k = 0;
    for (const char *p = text; *p && k + 1 < err_len; ++p) err[k++] = *p;
    if (detail) {
        for (const char *p = ": "; *p && k + 1 < err_len; ++p) err[k++] = *p;
        for (const char *p = detail; *p && k + 1 < err_len; ++p) err[k++] = *p;
    }
    err[k] = 0;
}

bool is_aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace
}  // namespace adama

extern "C" adama_status adama_linear_wgrad_fold_noalloc(
    const adama_config *cfg, int n_micro, const void *X, const void *dY, int tokens, int d_in,
    int d_out, int64_t ldx, int64_t ldy, float *m, float *v, int64_t ldmv, uint32_t *status_out_host,
    char *err, size_t err_len, void *cuda_stream) {
    using namespace adama;
    set_msg(err, err_len, "");
    if (!cfg || !(cfg->beta1 >= 0.0 && cfg->beta1 < 1.0) || !(cfg->beta2 >= 0.0 && cfg->beta2 < 1.0) ||
        cfg->device < 0 || (cfg->flags & ~ADAMA_GRADS_PRESCALED) != 0 || n_micro < 1) {
        set_msg(err, err_len, "noalloc: bad configuration or n_micro < 1");
        return ADAMA_ERR_INVALID_ARG;
    }
    if (cfg->device >= kMaxDevices) {
        set_msg(err, err_len, "noalloc: device ordinal beyond the 64 this entry point keeps set-up for");
        return ADAMA_ERR_UNSUPPORTED;
    }
    if (tokens < 0 || d_in < 1 || d_out < 1 || !m || !v || (tokens > 0 && (!X || !dY)) ||
        ldx < d_in || ldy < d_out || ldmv < d_out) {
        set_msg(err, err_len, "noalloc: bad shape, null pointer or row pitch smaller than the row");
        return ADAMA_ERR_INVALID_ARG;
    }
    if (!is_aligned(X, 16) || !is_aligned(dY, 16) || !is_aligned(m, 16) || !is_aligned(v, 16) ||
        ldx % 8 || ldy % 8 || ldmv % 4) {
        set_msg(err, err_len,
                "noalloc: X, dY, m, v must be 16-byte aligned, ldx and ldy multiples of 8, ldmv of 4");
        return ADAMA_ERR_MISALIGNED;
    }
    if (ldx * 2 >= (1ll << 40) || ldy * 2 >= (1ll << 40) || ldmv * 4 >= (1ll << 40)) {
        set_msg(err, err_len, "noalloc: row pitch too large for a tensor map");
        return ADAMA_ERR_UNSUPPORTED;
    }
    // Scratch the kernel would need for these shapes against what the static array holds.
    // The need is one status block for every shape, so this cannot fail today; it is
    // checked so that a later kernel with a shape-dependent need fails here, not on the GPU.
    const size_t scratch_needed = 256;
    if (scratch_needed > kStaticScratchBytes) {
        set_msg(err, err_len, "noalloc: problem needs more scratch than the 256-byte static block");
        return ADAMA_ERR_UNSUPPORTED;
    }

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
    cudaError_t e = (prev == cfg->device) ? cudaSuccess : cudaSetDevice(cfg->device);
    const char *msg = "cudaSetDevice";
    StaticSetup *setup = nullptr;
    if (e == cudaSuccess) e = static_setup_for_current_device(cfg->device, &setup, &msg);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (e == cudaSuccess && tokens > 0) {
        // every call shares the block, which still holds the last call's record
        msg = "cudaMemsetAsync(static scratch)";
        e = cudaMemsetAsync(setup->scratch, 0, kStaticScratchBytes, stream);
        if (e == cudaSuccess) {
            WgradArgs a;
            a.X = X;
            a.dY = dY;
            a.tokens = tokens;
            a.d_in = d_in;
            a.d_out = d_out;
            a.ldx = ldx;
            a.ldy = ldy;
            a.ldmv = ldmv;
            a.m = m;
            a.v = v;
            a.c = make_fold_constants(cfg->beta1, cfg->beta2, n_micro, cfg->flags);
            a.status = setup->scratch;
            a.sm_count = setup->sm_count;
            a.stream = stream;
            e = launch_wgrad_fold(a, &msg);
        }
        if (e == cudaSuccess && status_out_host) {
            msg = "cudaMemcpyAsync(status)";
            e = cudaMemcpyAsync(status_out_host, setup->scratch, 4 * sizeof(uint32_t),
                                cudaMemcpyDeviceToHost, stream);
        }
    } else if (e == cudaSuccess && status_out_host) {
        status_out_host[0] = status_out_host[1] = status_out_host[2] = status_out_host[3] = 0;
    }
    if (prev >= 0 && prev != cfg->device) cudaSetDevice(prev);
    if (e != cudaSuccess) {
        set_msg(err, err_len, msg, cudaGetErrorString(e));
        return ADAMA_ERR_CUDA;
    }
    return ADAMA_OK;
}
