// Internal declarations shared by the translation units of libadama (not installed).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "adama.h"

namespace adama {

// Constants of one mini-batch / one update, derived in double on the host and
// rounded to fp32 once (forming 1-beta2 in fp32 would already cost 1e-5
// relative accuracy on v).
struct FoldConstants {
    float a;  // (1-beta1)/N     (or 1-beta1 with ADAMA_GRADS_PRESCALED)
    float b;  // (1-beta2)/N^2   (or 1-beta2)
};

struct ApplyConstants {
    float step;      // lr / (1 - beta1^t)
    float inv_bc2;   // 1 / (1 - beta2^t)
    float eps;       // eps
    float beta1_hi;  // beta1 = beta1_hi + beta1_lo to ~1e-15: the decay m*beta1 is
    float beta1_lo;  // formed as fma(m, hi, m*lo), free of the per-step bias of a
    float beta2_hi;  // plain fp32 beta that would build up over ~1/(1-beta) steps
    float beta2_lo;
    float w_keep;    // 1 - lr*weight_decay (decoupled decay, AdamW); exactly 1 when it is off
};

// Coefficient statistics (Section 4.1): k = (1-beta2)/(1-beta1)^2 turns the squared change of m
// over a mini-batch into Adam's second-moment increment; beta2 = hi + lo as in ApplyConstants.
struct CoefConstants {
    float k;
    float beta2_hi;
    float beta2_lo;
};

// x = hi + lo with hi = fp32(x)
void split_hi_lo(double x, float *hi, float *lo);

FoldConstants make_fold_constants(double beta1, double beta2, int n_micro, unsigned flags);
// world > 1: m and v hold the SUM over `world` data-parallel ranks (Section 3.3 of the paper);
// the 1/world and 1/world^2 of Eqs. 6-7 and the world*beta2 pre-scaling of the next mini-batch
// are folded into the same constants, so the kernel is unchanged.
// sharded (ZeRO-style ownership): the caller's m, v are the owner's shard of the summed
// states and stay un-normalised between mini-batches (beta*sum instead of beta/R*sum),
// because the other ranks restart their accumulators for that shard from zero.
ApplyConstants make_apply_constants(double beta1, double beta2, double eps, int64_t t, double lr,
                                    int world = 1, bool sharded = false, double weight_decay = 0.0);

// Status block in device memory (256 bytes): word 0 = first error code recorded
// by a kernel (0 = none), word 1 = which wait, word 2 = tile; rest reserved.
enum DeviceErr : unsigned { kDevOk = 0, kDevTimeout = 1 };

// streaming kernels (fold_apply.cu)
cudaError_t launch_fold(const void *grad, adama_dtype gdt, float *m, float *v, size_t n,
                        FoldConstants c, int sm_count, cudaStream_t stream);
// w_bf16_out (may be null): n bf16 elements that receive the updated weights, rounded to nearest
cudaError_t launch_apply(float *w, float *m, float *v, size_t n, ApplyConstants c, int sm_count,
                         cudaStream_t stream, void *w_bf16_out = nullptr);

// SGD-momentum fold / apply and the coefficient statistics (extensions.cu)
cudaError_t launch_sgdm_fold(const void *grad, adama_dtype gdt, float *buf, size_t n, float inv_n,
                             int sm_count, cudaStream_t stream);
cudaError_t launch_sgdm_apply(float *w, float *buf, size_t n, float lr, float mu_hi, float mu_lo,
                              int sm_count, cudaStream_t stream);
// stats: 4 doubles in device memory {sum, min, max, count}; two launches (reset, pass)
cudaError_t launch_coefficient_stats(const float *m, const float *m_begin, const float *v,
                                     float *v_adam, size_t n, CoefConstants c, double *stats,
                                     int sm_count, cudaStream_t stream);

// multi-tensor forms (multi_tensor.cu): up to kMultiMax tensors per launch, each shorter than
// 2^32 * 4096 elements in total blocks
constexpr int kMultiMax = 64;
cudaError_t launch_fold_multi(const void *const *g, adama_dtype gdt, float *const *m,
                              float *const *v, const size_t *n, int count, FoldConstants c,
                              int sm_count, cudaStream_t stream);
cudaError_t launch_apply_multi(float *const *w, float *const *m, float *const *v, const size_t *n,
                               int count, ApplyConstants c, int sm_count, cudaStream_t stream);

// fused reduce-scatter + sharded apply + all-gather over peer-mapped buffers (peer_apply.cu)
constexpr int kMaxPeers = 16;
cudaError_t launch_apply_sharded_peers(float *const *w, float *const *m, float *const *v, int world,
                                       int rank, size_t n, ApplyConstants c, int sm_count,
                                       cudaStream_t stream);

// bias gradient (column sums of dY) + fold (bias_grad.cu)
cudaError_t launch_bias_grad_fold(const void *dY, int tokens, int d_out, int64_t ldy, float *m,
                                  float *v, FoldConstants c, cudaStream_t stream);

// fused weight-gradient + fold (wgrad_fold.cu)
// Which instance of the kernel a launch uses; 0 everywhere = chosen per launch from the shape.
// Set through adama_debug_set_wgrad_variant so that the tests reach every instance on every
// shape, whichever the automatic choice would be.
struct WgradVariant {
    int epilogue = 0;   // 1 = direct (accumulator -> registers -> m, v), 2 = staged through shared memory
    int epi_warps = 0;  // 4 or 8 epilogue warps (direct epilogue)
    int box_loads = 0;  // 1 = one TMA operation per 64-feature box even where grouped loads apply
    int no_pdl = 0;     // 1 = plain stream order instead of programmatic dependent launch
};
constexpr unsigned long long kDefaultWaitLimitNs = 2000000000ull;  // 2 s per device-side wait
struct WgradArgs {
    const void *X;
    const void *dY;
    int tokens, d_in, d_out;
    int64_t ldx, ldy, ldmv;
    float *m;
    float *v;
    FoldConstants c;
    unsigned *status;  // device status block
    int sm_count;
    cudaStream_t stream;
    // optional: moments of the layer's bias (d_out fp32 each); the column sums of dY are
    // folded into them by the same launch
    float *bias_m = nullptr;
    float *bias_v = nullptr;
    WgradVariant variant;
    unsigned long long wait_limit_ns = 0;  // 0 = kDefaultWaitLimitNs
    int withhold_last_load = 0;            // expiry test only: see adama_debug_wgrad_expire_wait
    int inputs_settled = 0;                // ADAMA_INPUTS_SETTLED: X, dY not written by the kernel just before
};
// Returns cudaSuccess or the failing CUDA error; *msg (static string) says which step failed.
cudaError_t launch_wgrad_fold(const WgradArgs &args, const char **msg);
// Several layers in ONE launch, worked through in the given order; stream, status block,
// constants, variant and wait limit are taken from layers[0].  1 <= count <= kMaxWgradLayers.
constexpr int kMaxWgradLayers = 8;
cudaError_t launch_wgrad_fold_multi(const WgradArgs *layers, int count, const char **msg);
// One-time, per process: resolves the driver's tensor-map encoder.
cudaError_t wgrad_fold_setup(const char **msg);
// Set-up bookkeeping, for diagnostics: bit 0 = the encoder has been resolved, bit 1 = the
// kernels' attributes have been set on `device`.
int wgrad_setup_state(int device);

}  // namespace adama
