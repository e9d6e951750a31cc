/*
 * adama.h -- C ABI of the B200 (sm_100a) AdamA optimizer library.
 *
 * AdamA (Adam Accumulation, arXiv 2305.19982) folds every micro-batch gradient
 * straight into the Adam moments, so the gradient can be dropped as soon as it
 * has been produced; at the end of the mini-batch a bias-corrected Adam update
 * is applied.  One mini-batch, in the order of the paper's Algorithm 2:
 *
 *     adama_begin_minibatch(ctx, N)            t <- t+1; fixes N
 *     for each micro-batch, for each layer (back to front):
 *         adama_linear_wgrad_fold(...)         linear layers: G = X^T.dY is folded
 *                                              from the tensor-core accumulator and
 *                                              never written to memory
 *         adama_fold(...)                      every other gradient tensor
 *     for each parameter tensor:
 *         adama_apply(...)                     update + beta-decay for the next step
 *
 * Conventions
 *   - All tensor pointers are DEVICE pointers unless a parameter is named
 *     *_host.  Memory is owned by the caller and only borrowed until the work
 *     queued on `cuda_stream` has completed.  The library allocates its context,
 *     a 256-byte device status block, one copy stream and a few events.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the default
 *     stream).  Calls are asynchronous and ordered by that stream.
 *   - Gradients are passed RAW (as autograd produces them for one micro-batch);
 *     the 1/N of Algorithm 2's "g <- (1/N) grad" is folded into the
 *     coefficients a = (1-beta1)/N and b = (1-beta2)/N^2.  With the flag
 *     ADAMA_GRADS_PRESCALED the caller has already divided by N and the
 *     coefficients are a = 1-beta1, b = 1-beta2.
 *   - State convention: Algorithm 2 decays m and v at the START of a
 *     mini-batch.  This library performs that decay at the END of the previous
 *     one, inside adama_apply, which stores beta1*m_t and beta2*v_t.  With
 *     m_0 = v_0 = 0 the two orders give identical m_t, v_t and theta_t.  Between
 *     adama_apply and the next fold the buffers therefore hold the decayed
 *     moments; between the last fold and adama_apply they hold m_t and v_t.
 *   - Hyper-parameters are doubles; every derived constant (1-beta, 1-beta^t,
 *     lr/(1-beta1^t), ...) is formed in double on the host and rounded to fp32
 *     once.
 *   - One context per model replica.  A context is not thread-safe.
 *   - Every function returns an adama_status; nothing aborts, traps or prints.
 *     adama_last_error gives a message for the last failing call on a context.
 */
#ifndef ADAMA_H_
#define ADAMA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define ADAMA_API __attribute__((visibility("default")))
#else
#define ADAMA_API
#endif

typedef struct adama_ctx adama_ctx; /* opaque; created by adama_init, freed by adama_destroy */

typedef enum adama_status {
    ADAMA_OK = 0,
    ADAMA_ERR_INVALID_ARG = 1, /* null pointer, negative size, N < 1, bad hyper-parameter      */
    ADAMA_ERR_BAD_STATE = 2,   /* call order: fold/apply before the first begin_minibatch      */
    ADAMA_ERR_MISALIGNED = 3,  /* pointer or pitch violates the alignment stated for the call  */
    ADAMA_ERR_UNSUPPORTED = 4, /* device is not sm_100, or a size exceeds a documented limit   */
    ADAMA_ERR_CUDA = 5,        /* a CUDA runtime/driver call failed; see adama_last_error      */
    ADAMA_ERR_TIMEOUT = 6      /* a bounded device-side wait expired (reported by sync_status) */
} adama_status;

typedef enum adama_dtype { ADAMA_F32 = 0, ADAMA_BF16 = 1 } adama_dtype;

/* flags for adama_config.flags */
#define ADAMA_GRADS_PRESCALED 1u /* gradients already carry the 1/N of Algorithm 2 */
/* adama_apply_to_host copies the weights back on a stream of the context's own instead of on
 * `cuda_stream`, so that the copy (device to host) can run while later calls already stream the
 * next gradients in (host to device); see adama_apply_to_host for what the caller gives up. */
#define ADAMA_ASYNC_COPYBACK 2u
/* Promise about the inputs of the fused weight-gradient calls (adama_linear_wgrad_fold, _bias_fold,
 * _multi): the X and dY handed to a call are NOT written by the kernel enqueued just before the
 * call on the same stream -- they were complete earlier, as in a deferred weight-gradient pass or
 * when the producing kernel is followed by some other kernel first.  The call's operand loads then
 * do not wait for that previous kernel, so its first tiles run while the previous call's last,
 * partly filled round of tiles still finishes (back-to-back calls on 1600 x 1600, 4096 tokens:
 * 34.9 -> 22.5 us).  Everything else keeps its order: m, v (and the bias moments and dY reads of
 * the bias warps) are touched only after the previous kernel has completed, so consecutive calls
 * on the same layer stay correct.  Without the flag, the default, nothing is assumed. */
#define ADAMA_INPUTS_SETTLED 4u

typedef struct adama_config {
    double beta1;   /* in [0,1)                                    */
    double beta2;   /* in [0,1)                                    */
    double eps;     /* >= 0; added outside the square root         */
    int device;     /* CUDA device ordinal the context is bound to */
    unsigned flags; /* ADAMA_* flags                               */
} adama_config;

/* Algorithm 2, "Initialize": t <- 0.  (theta_0, m_0 = 0 and v_0 = 0 are the
 * caller's buffers: the caller zero-fills m and v once.)  Creates the context
 * on cfg->device, which must be a compute-capability-10.x GPU; the device's
 * primary context is initialised if needed.  Allocates a 256-byte device
 * status block, a copy stream and a few events.
 * Errors: INVALID_ARG (null, betas outside [0,1), eps < 0), UNSUPPORTED (not
 * sm_100), CUDA. */
ADAMA_API adama_status adama_init(adama_ctx **out, const adama_config *cfg);

/* Frees everything adama_init allocated.  The caller must have synchronised
 * the streams it used.  NULL is accepted. */
ADAMA_API adama_status adama_destroy(adama_ctx *ctx);

/* Algorithm 2, first line of the loop body: t <- t+1, and N (micro-batches in
 * this mini-batch, >= 1) is fixed, which fixes a = (1-beta1)/N and
 * b = (1-beta2)/N^2 for every fold until the next call.  Host-only, no GPU
 * work: the decay "m <- beta1 m, v <- beta2 v" of the same line was already
 * applied by the previous adama_apply (see "State convention").
 * Errors: INVALID_ARG (n_micro < 1). */
ADAMA_API adama_status adama_begin_minibatch(adama_ctx *ctx, int n_micro);

/* Algorithm 2, inner loop body for one (micro-batch, layer):
 *     m <- m + (1-beta1) g,   v <- v + (1-beta2) g^2,   g = grad / N
 * computed as m += a*grad, v += b*grad^2 in fp32 (one FMA each).
 *   grad : n elements, dtype gdt (fp32 or bf16), contiguous, device, read-only
 *   m, v : n fp32 elements each, contiguous, device, updated in place
 * Any n >= 0 and any element-aligned pointers are accepted: the kernel uses
 * 128-bit accesses when grad, m and v allow it and a scalar path otherwise.
 * m and v must not overlap each other or grad.
 * Errors: INVALID_ARG, BAD_STATE (no begin_minibatch yet), MISALIGNED (pointer
 * not aligned to its element size), CUDA (launch failure). */
ADAMA_API adama_status adama_fold(adama_ctx *ctx, const void *grad, adama_dtype gdt, float *m,
                                  float *v, size_t n, void *cuda_stream);

/* The same accumulation for a linear layer y = x.W, W of shape [d_in, d_out],
 * whose raw weight gradient is G = X^T.dY (Section 3.1 folds a layer's gradient
 * into the moments as soon as backward has produced it; the buffer that Algorithm 2
 * assigns and releases for it disappears because G only ever exists as a
 * tensor-memory accumulator tile):
 *     G[p,q] = sum_{tau < tokens} X[tau,p] * dY[tau,q]   (bf16 x bf16 -> fp32)
 *     m[p,q] += a*G[p,q],   v[p,q] += b*G[p,q]^2
 *   X    : [tokens, d_in]  bf16 row-major, row pitch ldx  elements, device, read-only
 *   dY   : [tokens, d_out] bf16 row-major, row pitch ldy  elements, device, read-only
 *   m, v : [d_in, d_out]   fp32 row-major, row pitch ldmv elements, device, in place
 * Requirements (checked, MISALIGNED / INVALID_ARG otherwise): X, dY, m, v
 * 16-byte aligned; ldx, ldy multiples of 8; ldmv a multiple of 4; ldx >= d_in,
 * ldy >= d_out, ldmv >= d_out; d_in, d_out >= 1; tokens >= 0 (0 is a no-op).
 * Any d_in, d_out, tokens within those rules are handled (ragged tiles are
 * zero-filled on load and clipped on store).  The whole token sum of one call
 * is finished before it is squared: there is no split over tokens.
 * m and v are read, updated with one fma per element and written back by the
 * kernel's epilogue; each element is touched by exactly one tile per call, so
 * results do not depend on scheduling.
 * A caller that stores W as [d_out, d_in] passes (dY, X) in place of (X, dY).
 * Device-side waits are bounded; if one expires the kernel stops early, leaves
 * a code in the status block and adama_sync_status returns ADAMA_ERR_TIMEOUT.
 * Errors: INVALID_ARG, BAD_STATE, MISALIGNED, UNSUPPORTED, CUDA. */
ADAMA_API adama_status adama_linear_wgrad_fold(adama_ctx *ctx, const void *X, const void *dY,
                                               int tokens, int d_in, int d_out, int64_t ldx,
                                               int64_t ldy, float *m, float *v, int64_t ldmv,
                                               void *cuda_stream);

/* adama_linear_wgrad_fold for several layers in as few launches as possible (at most 8 layers per
 * launch), e.g. the linear layers of one transformer block whose (X, dY) pairs backward has
 * produced.  Per layer it computes exactly what adama_linear_wgrad_fold (or, where m_bias and
 * v_bias are given, adama_linear_wgrad_bias_fold) computes, bit for bit: Algorithm 2's inner
 * loop body for layer j, for the `count` layers in the order given.  What changes is the
 * schedule: the layers' tiles form one work list, so the CTA pairs that a layer's last round
 * of tiles leaves idle start on the next layer, the epilogue of a layer's last tile overlaps
 * the next layer's first main loop, and kernel set-up, pipeline fill and the final exposed
 * epilogue are paid once per launch instead of once per layer.  The price is that the layers'
 * X and dY must all be alive until the launch has run (they can be released one launch later
 * than with per-layer calls; m, v and the weight gradient are unaffected: there still is no
 * gradient buffer).  The layers must not share m or v storage, and no X or dY may overlap any
 * layer's m, v or bias moments.  A call with more than 8 layers makes several launches; from its
 * second launch on the operand loads do not wait for the call's own previous launch (which
 * writes no X or dY), so consecutive launches overlap at their seams as with
 * ADAMA_INPUTS_SETTLED.
 *   items : `count` descriptions in HOST memory, read before the call returns; per item the
 *           arguments of adama_linear_wgrad_fold, plus m_bias / v_bias (both null or both set).
 * Items with tokens == 0 are skipped.  Errors: as adama_linear_wgrad_fold, reported for the
 * first offending item before anything is launched. */
typedef struct adama_linear_item {
    const void *X;
    const void *dY;
    int tokens, d_in, d_out;
    int64_t ldx, ldy;
    float *m;
    float *v;
    int64_t ldmv;
    float *m_bias; /* may be null (then v_bias must be null too) */
    float *v_bias;
} adama_linear_item;
ADAMA_API adama_status adama_linear_wgrad_fold_multi(adama_ctx *ctx, const adama_linear_item *items,
                                                     int count, void *cuda_stream);

/* adama_linear_wgrad_fold that also folds the layer's bias gradient, the column sums of dY,
 *     g[q] = sum_{tau < tokens} dY[tau,q],   m_bias[q] += a*g[q],   v_bias[q] += b*g[q]^2
 * (Algorithm 2, inner loop body, for the bias of the same layer) in the same launch: two
 * extra warps per CTA read dY from global memory (it is L2-resident: the producer is loading
 * the same data) and form the sums while the other roles run the tiles; every 32-column slab
 * is summed over all tokens by one CTA, so the sum is complete before it is squared, and the
 * result is deterministic.
 *   m_bias, v_bias : d_out fp32 elements each, contiguous, device, updated in place.
 * Weight results are bit-identical to adama_linear_wgrad_fold; the bias results equal
 * adama_bias_grad_fold's up to the order of the fp32 token sum.
 * Errors: as adama_linear_wgrad_fold, plus INVALID_ARG (null bias moments), MISALIGNED. */
ADAMA_API adama_status adama_linear_wgrad_bias_fold(adama_ctx *ctx, const void *X, const void *dY,
                                                    int tokens, int d_in, int d_out, int64_t ldx,
                                                    int64_t ldy, float *m, float *v, int64_t ldmv,
                                                    float *m_bias, float *v_bias,
                                                    void *cuda_stream);

/* Algorithm 2, "Update", fused with the first line of the NEXT loop body:
 *     m_hat = m/(1-beta1^t), v_hat = v/(1-beta2^t),
 *     w <- w - lr * m_hat / (sqrt(v_hat) + eps)
 *     m <- beta1*m, v <- beta2*v            (decay for mini-batch t+1)
 *   w, m, v : n fp32 elements each, contiguous, device, updated in place.
 * `lr` is the step size alpha of this mini-batch (schedules stay with the
 * caller).  Call once per parameter tensor per mini-batch, after its last fold.
 * Errors: INVALID_ARG, BAD_STATE (t == 0), MISALIGNED, CUDA. */
ADAMA_API adama_status adama_apply(adama_ctx *ctx, float *w, float *m, float *v, size_t n,
                                   double lr, void *cuda_stream);

/* adama_apply that also writes the updated weights rounded to bf16 (round to nearest even)
 * into w_bf16_out (n bf16 elements, device): the copy a mixed-precision forward pass reads,
 * produced in the same pass (26 B/param) instead of by a separate cast (24 + 6).  The fp32
 * w stays the master copy; w, m, v results are bit-identical to adama_apply.
 * Errors: as adama_apply, plus INVALID_ARG (null output), MISALIGNED. */
ADAMA_API adama_status adama_apply_bf16_copy(adama_ctx *ctx, float *w, float *m, float *v,
                                             void *w_bf16_out, size_t n, double lr,
                                             void *cuda_stream);

/* The bias of the same linear layer: its raw micro-batch gradient is the column sum of dY,
 *     g[q] = sum_{tau < tokens} dY[tau,q],   m[q] += a*g[q],   v[q] += b*g[q]^2
 * (Algorithm 2, inner loop body; the sum over tokens is completed on-chip, by a cluster of
 * CTAs through distributed shared memory, before it is squared).  dY as in
 * adama_linear_wgrad_fold (bf16, row pitch ldy, 16-byte aligned, ldy a multiple of 8);
 * m, v: d_out fp32 elements each, contiguous.  tokens == 0 is a no-op.  Deterministic.
 * Errors: INVALID_ARG, BAD_STATE, MISALIGNED, CUDA. */
ADAMA_API adama_status adama_bias_grad_fold(adama_ctx *ctx, const void *dY, int tokens, int d_out,
                                            int64_t ldy, float *m, float *v, void *cuda_stream);

/* adama_fold for a list of tensors in as few launches as possible (Algorithm 2's inner loop
 * visits "each layer"; a transformer has hundreds of small ones: biases, norm scales).
 * grads, m, v, n are HOST arrays of `count` entries: device pointers and element counts; all
 * gradients share the dtype gdt.  Tensors shorter than 4 Mi elements are grouped, up to 64
 * per launch, the table travelling in the kernel's parameters (nothing is allocated); longer
 * ones get the single-tensor kernel.  Same arithmetic and the same per-tensor rules as
 * adama_fold; results are bit-identical to `count` adama_fold calls.  The arrays are read
 * before the call returns.  Errors: as adama_fold, for the first offending tensor. */
ADAMA_API adama_status adama_fold_multi(adama_ctx *ctx, const void *const *grads, adama_dtype gdt,
                                        float *const *m, float *const *v, const size_t *n,
                                        int count, void *cuda_stream);

/* adama_apply for a list of tensors, grouped like adama_fold_multi; bit-identical to `count`
 * adama_apply calls with the same lr. */
ADAMA_API adama_status adama_apply_multi(adama_ctx *ctx, float *const *w, float *const *m,
                                         float *const *v, const size_t *n, int count, double lr,
                                         void *cuda_stream);

/* Data-parallel variant of adama_apply (Section 3.3, Eqs. 4-7): R = world_size devices
 * each fold their own N micro-batches into their own m and v; once per mini-batch the
 * CALLER sums m and v over the devices (one all-reduce each, e.g. NCCL, on the same
 * stream order); this call then takes the summed buffers and computes
 *     m_t = m/R,  v_t = v/R^2                          (the paper's averaging of the states)
 *     w <- w - lr * (m_t/(1-beta1^t)) / (sqrt(v_t/(1-beta2^t)) + eps)
 *     m <- beta1*m_t,  v <- R*beta2*v_t                (Section 3.3: v decays by devices*beta2, Eq. 5)
 * so that R devices x N micro-batches give exactly the update of one device with N*R
 * micro-batches.  Every rank calls it with the same arguments and ends with the same w.
 * Between mini-batches each rank's v therefore holds R*beta2*v_t (m holds beta1*m_t).
 * world_size == 1 is adama_apply.  All scalings are folded, in double, into the
 * constants of the same kernel.  Errors as adama_apply, plus INVALID_ARG (world_size < 1). */
ADAMA_API adama_status adama_apply_allreduced(adama_ctx *ctx, float *w, float *m, float *v,
                                              size_t n, double lr, int world_size,
                                              void *cuda_stream);

/* State-sharded variant: the paper combines AdamA with ZeRO-DP P_os (Section 4.2, "Memory
 * Reduction") but prints no algorithm for it; this is this library's construction on top of
 * Section 3.3, chosen so that Eqs. 6-7 still hold.  Rank r owns one contiguous shard of every parameter buffer.  Each rank still
 * folds full-size local accumulators m, v; once per mini-batch the CALLER reduce-scatters
 * (sums) them so that the owner holds the summed shard, calls this function on its shard of
 * w, m, v, zero-fills the shards of m and v it does not own, and all-gathers w.  With
 * S_m, S_v the summed shard:
 *     m_t = S_m/R,  v_t = S_v/R^2,  w <- w - lr * (m_t/(1-beta1^t)) / (sqrt(v_t/(1-beta2^t)) + eps)
 *     m <- beta1*S_m (= R*beta1*m_t),  v <- beta2*S_v (= R^2*beta2*v_t)
 * The un-normalised storage is what makes the next mini-batch's sum come out right when the
 * non-owners restart from zero: (beta2*S_v + new folds)/R^2 = beta2*v_t + ... (Eq. 7).
 * Persistent optimizer state per rank is 1/R of m and v.  Errors as adama_apply_allreduced. */
ADAMA_API adama_status adama_apply_sharded(adama_ctx *ctx, float *w, float *m, float *v, size_t n,
                                           double lr, int world_size, void *cuda_stream);

/* adama_apply_sharded with the exchange fused into the kernel: no separate reduce-scatter or
 * all-gather.  w_peers, m_peers, v_peers are HOST arrays of world_size device pointers: entry
 * q is rank q's full-size buffer (n fp32 elements), mapped into this process's address space
 * (peer access over NVLink: IPC handles or symmetric memory; entry `rank` is the local one).
 * This rank's launch reads shard `rank` (elements [rank*n/R, (rank+1)*n/R)) of every rank's m
 * and v with plain loads, sums them in rank order, updates its shard of w as
 * adama_apply_sharded does, and writes: the un-normalised sums into its own m, v shard, zeros
 * into that shard of every other rank's m, v, and the new weights into that shard of every
 * rank's w.  Shard r of all buffers is touched by rank r's launch only, and the kernel never
 * waits for a peer.  The CALLER orders it against the folds: every rank has finished folding
 * before the first of these launches starts, and none folds (or reads w) again before all of
 * them have finished.  n must be a multiple of 4*world_size, all buffers 16-byte aligned,
 * world_size <= 16.  Errors: INVALID_ARG, BAD_STATE, MISALIGNED, UNSUPPORTED, CUDA. */
ADAMA_API adama_status adama_apply_sharded_peers(adama_ctx *ctx, float *const *w_peers,
                                                 float *const *m_peers, float *const *v_peers,
                                                 int world_size, int rank, size_t n, double lr,
                                                 void *cuda_stream);

/* ---- host-buffer variants (same arithmetic, copies included) --------------------------- */

/* adama_fold with the gradient in HOST memory (pinned memory for full copy
 * speed).  The gradient is streamed through `staging` (device, caller-owned,
 * staging_bytes >= 2 MiB, 256-byte aligned) in two alternating halves on the
 * context's copy stream while the fold of the previous half runs on
 * `cuda_stream`.  On return all work is queued; grad_host and staging are
 * borrowed until `cuda_stream` has completed. */
ADAMA_API adama_status adama_fold_host(adama_ctx *ctx, const void *grad_host, adama_dtype gdt,
                                       float *m, float *v, size_t n, void *staging,
                                       size_t staging_bytes, void *cuda_stream);

/* adama_linear_wgrad_fold with X and dY in HOST memory, dense (ldx = d_in,
 * ldy = d_out, both multiples of 8).  Both are copied into `staging` (device,
 * caller-owned, at least 2*tokens*(d_in+d_out) + 256 bytes, 256-byte aligned)
 * on `cuda_stream`, then the fused kernel runs. */
ADAMA_API adama_status adama_linear_wgrad_fold_host(adama_ctx *ctx, const void *X_host,
                                                    const void *dY_host, int tokens, int d_in,
                                                    int d_out, float *m, float *v, int64_t ldmv,
                                                    void *staging, size_t staging_bytes,
                                                    void *cuda_stream);

/* adama_apply followed by a device-to-host copy of the updated weights into
 * w_host (n fp32, pinned memory for full speed), queued on `cuda_stream`.
 * With ADAMA_ASYNC_COPYBACK the copy is queued on the context's copy-back stream instead,
 * after the update: `cuda_stream` does not wait for it, so the host-to-device copies of
 * later *_host calls overlap it (the two directions of the link run at once).  The caller
 * then must not write w, nor read w_host, until one of these has happened on this context:
 * the next adama_apply* / adama_sgdm_apply call (it makes its stream wait for the copy),
 * or adama_sync_status (it returns after the copy has finished). */
ADAMA_API adama_status adama_apply_to_host(adama_ctx *ctx, float *w, float *m, float *v, size_t n,
                                           double lr, float *w_host, void *cuda_stream);

/* ---- for callers that must not allocate ------------------------------------------------- */

/* The paper has no counterpart to this call; it exists for integration reasons only.
 *
 * Same computation as adama_linear_wgrad_fold, for code that is not allowed to take device
 * memory from CUDA: for example a training job whose whole GPU memory is owned by a
 * framework's pool, or a component that runs while the allocator must stay untouched.
 * Such code cannot call adama_init (it allocates the status block), so this function takes
 * the hyper-parameters and N directly and needs no context: a = (1-beta1)/N and
 * b = (1-beta2)/N^2 are derived from cfg and n_micro exactly as a context would.
 *
 * The only memory the kernel uses besides X, dY, m and v is its 256-byte status block.
 * Here that block is a fixed array inside the library image: every GPU that loads the
 * library holds those 256 bytes until the process exits.  256 bytes is also the most this
 * entry point can ever provide; a shape whose kernel needed more would be refused with
 * ADAMA_ERR_UNSUPPORTED (today the need is the same for every shape).  The function calls
 * no cudaMalloc/cudaFree and no allocating library routine.
 *
 *   - The first call on each device looks the array's device address up and sets the
 *     kernel's shared-memory limit.  Make that first call outside any stream capture.
 *   - All calls, from all threads and streams, share the one block.  It is cleared on the
 *     stream before each launch.  Two calls that run on the GPU at the same time race on
 *     it: the arithmetic on m and v stays correct, but a recorded time-out may be lost or
 *     attributed to the wrong call.  Order such calls on one stream if the record matters.
 *   - status_out_host (may be NULL): 4 words of host memory (pinned, if the copy is to be
 *     asynchronous) that receive, once the stream reaches that point, {code, wait, tile, 0};
 *     code 0 = finished normally, 1 = a bounded device-side wait expired.
 *   - err / err_len (may be NULL / 0): caller's buffer for a message when the result is not
 *     ADAMA_OK.
 * Arguments X .. ldmv and their alignment rules are those of adama_linear_wgrad_fold.
 * Errors: INVALID_ARG, MISALIGNED, UNSUPPORTED (device ordinal >= 64, pitch too large,
 * scratch need above 256 bytes), CUDA. */
ADAMA_API adama_status adama_linear_wgrad_fold_noalloc(
    const adama_config *cfg, int n_micro, const void *X, const void *dY, int tokens, int d_in,
    int d_out, int64_t ldx, int64_t ldy, float *m, float *v, int64_t ldmv,
    uint32_t *status_out_host, char *err, size_t err_len, void *cuda_stream);

/* ---- beside the paper's algorithms ------------------------------------------------------ */

/* SGD with momentum on Algorithm 2's pipeline (the paper's Discussion remarks that other
 * momentum optimizers can take the same accumulation; the paper gives no algorithm for it):
 *     buf_t = mu*buf_{t-1} + sum_i grad_i/N,     w_t = w_{t-1} - lr*buf_t.
 * adama_sgdm_fold adds one raw micro-batch gradient:  buf <- buf + grad/N  (N from
 * adama_begin_minibatch; grad/1 under ADAMA_GRADS_PRESCALED), so no gradient buffer outlives
 * the layer's backward step.  adama_sgdm_apply does  w <- w - lr*buf  and then stores
 * buf <- mu*buf, the decay of the NEXT mini-batch (the same convention as adama_apply).
 *   grad : n elements of gdt, device, read-only;  buf, w : n fp32, device, in place.
 * 16-byte aligned pointers (8 for bf16 grad) take the 128-bit path, others a scalar one.
 * Errors: INVALID_ARG (null pointer, dtype, lr not finite, momentum outside [0,1)), BAD_STATE
 * (no adama_begin_minibatch yet), MISALIGNED, CUDA. */
ADAMA_API adama_status adama_sgdm_fold(adama_ctx *ctx, const void *grad, adama_dtype gdt,
                                       float *buf, size_t n, void *cuda_stream);
ADAMA_API adama_status adama_sgdm_apply(adama_ctx *ctx, float *w, float *buf, size_t n, double lr,
                                        double momentum, void *cuda_stream);

/* Section 4.1, the coefficient between AdamA's and standard Adam's adaptive scaling,
 *     c = sqrt(v_hat_t) / sqrt(v_hat_t'),
 * v_hat AdamA's bias-corrected second moment and v_hat' the one standard Adam would hold on
 * the same gradients (Algorithm 1, the first bracket term).  The paper plots the mean of c over
 * the elements and its range per training step; this call produces those three numbers.
 * Call it after the mini-batch's last fold and BEFORE adama_apply:
 *   m, v    : the AdamA states as they stand (n fp32 each, device, read-only);
 *   m_begin : copy of m taken right after adama_begin_minibatch, before the first fold (n fp32,
 *             device, read-only); NULL means all zeros (the first mini-batch).  The mini-batch
 *             gradient sum is recovered from it, (m - m_begin)/(1-beta1) = sum_i grad_i/N, so the
 *             fused weight-gradient path needs no gradient buffer for this either;
 *   v_adam  : Adam's second moment, n fp32, device, updated in place.  It follows the
 *             convention of v: on entry beta2*v'_{t-1} (zeros before the first mini-batch), on
 *             exit beta2*v'_t;
 *   stats_dev : 4 doubles in DEVICE memory, 8-byte aligned, overwritten on the stream with
 *             {sum of c, min c, max c, number of elements counted}; mean = sum/count.
 * Elements whose v'_t is zero have no coefficient and are not counted; with none counted
 * min is +infinity and max is 0.  The bias corrections of v_hat and v_hat' are equal and
 * cancel.  Two launches (reset of stats, one pass of 20 B/element).  The sum is formed with
 * double atomics, so its last bits may differ from run to run.
 * Errors: INVALID_ARG, BAD_STATE (no adama_begin_minibatch yet), MISALIGNED, CUDA. */
ADAMA_API adama_status adama_coefficient_stats(adama_ctx *ctx, const float *m, const float *m_begin,
                                               const float *v, float *v_adam, size_t n,
                                               double *stats_dev, void *cuda_stream);

/* ---- state, checkpointing, diagnostics ------------------------------------------------- */

/* Step counter t of Algorithm 2 (0 after init). */
ADAMA_API int64_t adama_get_step(const adama_ctx *ctx);
/* Restore t from a checkpoint (t >= 0).  The saved m, v must follow the state
 * convention above (decayed if saved after adama_apply). */
ADAMA_API adama_status adama_set_step(adama_ctx *ctx, int64_t t);
/* Micro-batch count fixed by the last begin_minibatch (0 before the first). */
ADAMA_API int adama_get_n_micro(const adama_ctx *ctx);

/* Extension beyond the paper's algorithms (its Discussion notes that other momentum-based
 * optimizers can use the same accumulation): decoupled weight decay as in AdamW.  With
 * weight_decay = lambda > 0 every later apply computes
 *     w <- w*(1 - lr*lambda) - lr * m_hat / (sqrt(v_hat) + eps)
 * (the decay is not folded into m or v).  lambda = 0, the default, is Algorithm 2 exactly
 * (the factor is 1.0f, results are bit-identical).  Errors: INVALID_ARG (negative or not finite). */
ADAMA_API adama_status adama_set_weight_decay(adama_ctx *ctx, double weight_decay);

/* Waits for `cuda_stream`, then reads and clears the device status block.
 * Returns ADAMA_OK, ADAMA_ERR_TIMEOUT (a bounded wait inside the fused kernel
 * expired; m and v of that call are incomplete) or ADAMA_ERR_CUDA. */
ADAMA_API adama_status adama_sync_status(adama_ctx *ctx, void *cuda_stream);

/* Test hook: writes {code, wait, tile} into the device status block exactly as a kernel whose
 * bounded wait expired would, so that the host side of the time-out path (adama_sync_status:
 * report, message, clearing, continued use of the context) can be exercised without making
 * any kernel wait in vain.  Synchronises `cuda_stream`. */
ADAMA_API adama_status adama_debug_set_status(adama_ctx *ctx, unsigned code, unsigned wait,
                                              unsigned tile, void *cuda_stream);

/* Test hook: makes a device-side wait of the fused weight-gradient kernel actually run out, in
 * the non-hanging form.  Launches the kernel of adama_linear_wgrad_fold (same arguments, same
 * checks) with every bounded wait limited to `wait_limit_ns` (>= 1000, <= 10^9) instead of
 * 2 s, and with the producer told not to load the last 64-token stage of the launch's last
 * tile.  The issuer's wait for that stage expires; it records {time-out, which wait, tile} in
 * the status block, every role of the CTA pair gives up within its own limit, issued MMAs and
 * loads are waited for, tensor memory is released and the kernel returns.  All other tiles of
 * the launch are folded normally; the last tile's m, v are left untouched.  The following
 * adama_sync_status returns ADAMA_ERR_TIMEOUT and clears the block; the context stays usable.
 * No wait in the kernel is unbounded and nothing faults.  Errors: as adama_linear_wgrad_fold,
 * plus INVALID_ARG for a limit out of range or tokens == 0. */
ADAMA_API adama_status adama_debug_wgrad_expire_wait(adama_ctx *ctx, const void *X, const void *dY,
                                                     int tokens, int d_in, int d_out, int64_t ldx,
                                                     int64_t ldy, float *m, float *v, int64_t ldmv,
                                                     uint64_t wait_limit_ns, void *cuda_stream);

/* Test hook: pins which instance of the fused weight-gradient kernel this context launches, so
 * that every instance can be checked on every shape whatever the automatic choice would be.
 * 0 = automatic (the default).  epilogue: 1 = direct, 2 = staged through shared memory;
 * epi_warps: 4 or 8 (direct epilogue); box_loads: 1 = one TMA operation per 64-feature box
 * even where grouped loads apply; no_pdl: 1 = plain stream order instead of programmatic
 * dependent launch.
 * Results do not depend on the choice beyond fp32 summation order inside the tensor cores
 * (none: the order over tokens is the same).  Errors: INVALID_ARG for any other value. */
ADAMA_API adama_status adama_debug_set_wgrad_variant(adama_ctx *ctx, int epilogue, int epi_warps,
                                                     int box_loads, int no_pdl);

/* Diagnostics of the library's one-time set-up: bit 0 = the driver's tensor-map encoder has been
 * resolved (once per process), bit 1 = the fused kernel's attributes have been set on `device`
 * (once per device: a process that uses several GPUs sets each of them up at its first launch
 * there).  Needs no GPU. */
ADAMA_API int adama_debug_setup_state(int device);

/* Message for the most recent non-OK status returned on this context ("" if
 * none).  The pointer stays valid until the next call on the context. */
ADAMA_API const char *adama_last_error(const adama_ctx *ctx);

/* Number of kernels this context has launched since adama_init. */
ADAMA_API int64_t adama_launch_count(const adama_ctx *ctx);

/* Host-only, no GPU needed: the fp32 constants the kernels receive for a given
 * configuration, N, step t (>= 1) and lr, each derived in double from
 * Algorithm 2 and rounded once:
 *   out[0] = a = (1-beta1)/N          out[1] = b = (1-beta2)/N^2
 *   out[2] = lr/(1-beta1^t)           out[3] = 1/(1-beta2^t)        out[4] = eps
 *   out[5], out[6] = beta1 split as hi + lo   out[7], out[8] = beta2 split as hi + lo
 * Errors: INVALID_ARG. */
ADAMA_API adama_status adama_host_constants(const adama_config *cfg, int n_micro, int64_t t,
                                            double lr, float out[9]);

/* The same for adama_apply_allreduced with world_size R: out[2] = lr/(1-beta1^t)/R,
 * out[3] = 1/(1-beta2^t)/R^2, out[5..6] = beta1/R as hi + lo, out[7..8] = beta2/R as hi + lo. */
ADAMA_API adama_status adama_host_constants_allreduced(const adama_config *cfg, int n_micro,
                                                       int64_t t, double lr, int world_size,
                                                       float out[9]);

/* The same for adama_apply_sharded: as _allreduced, but out[5..6] = beta1 and out[7..8] = beta2
 * (hi + lo), since the owner keeps the un-normalised sums. */
ADAMA_API adama_status adama_host_constants_sharded(const adama_config *cfg, int n_micro,
                                                    int64_t t, double lr, int world_size,
                                                    float out[9]);

/* Library version, "major.minor.patch". */
ADAMA_API const char *adama_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ADAMA_H_ */
