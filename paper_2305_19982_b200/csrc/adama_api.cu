// C ABI of libadama: context, argument checks, host-side constants, launches.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <new>

#include "adama_internal.h"

struct adama_ctx {
    adama_config cfg;
    int64_t t;    // step counter of Algorithm 2
    int n_micro;  // N of the current mini-batch (0 before the first)
    adama::FoldConstants fold_c;
    int sm_count;
    unsigned *status_dev;      // 256-byte device status block
    cudaStream_t copy_stream;  // host-buffer variants: H2D copies overlap the folds
    cudaStream_t d2h_stream;   // ADAMA_ASYNC_COPYBACK: weights go back to the host here
    cudaEvent_t ev_applied, ev_d2h_done;
    bool d2h_pending;          // a copy-back that no stream has been made to wait for yet
    cudaEvent_t ev_copied[2], ev_folded[2], ev_entry;
    int64_t launches;
    double weight_decay;  // decoupled (AdamW) decay; 0 = the paper's plain update
    adama::WgradVariant variant;  // adama_debug_set_wgrad_variant; all 0 = automatic
    char err[256];
};

namespace adama {

FoldConstants make_fold_constants(double beta1, double beta2, int n_micro, unsigned flags) {
    double N = (flags & ADAMA_GRADS_PRESCALED) ? 1.0 : (double)n_micro;
    FoldConstants c;
    c.a = (float)((1.0 - beta1) / N);
    c.b = (float)((1.0 - beta2) / (N * N));
    return c;
}

void split_hi_lo(double x, float *hi, float *lo) {
    *hi = (float)x;
    *lo = (float)(x - (double)*hi);
}

ApplyConstants make_apply_constants(double beta1, double beta2, double eps, int64_t t, double lr,
                                    int world, bool sharded, double weight_decay) {
    ApplyConstants c;
    const double R = (double)world;
    double bc1 = 1.0 - pow(beta1, (double)t);
    double bc2 = 1.0 - pow(beta2, (double)t);
    // m_t = m/R, v_t = v/R^2 (Eqs. 6-7); w -= lr * (m_t/bc1) / (sqrt(v_t/bc2) + eps)
    c.step = (float)(lr / bc1 / R);
    c.inv_bc2 = (float)(1.0 / bc2 / (R * R));
    c.eps = (float)eps;
    c.w_keep = (float)(1.0 - lr * weight_decay);
    // stored for the next mini-batch: beta1*m_t = (beta1/R)*m and R*beta2*v_t = (beta2/R)*v
    // (sharded: the owner keeps R*beta1*m_t = beta1*m and R^2*beta2*v_t = beta2*v)
    split_hi_lo(sharded ? beta1 : beta1 / R, &c.beta1_hi, &c.beta1_lo);
    split_hi_lo(sharded ? beta2 : beta2 / R, &c.beta2_hi, &c.beta2_lo);
    return c;
}

}  // namespace adama

namespace {

adama_status fail(adama_ctx *ctx, adama_status st, const char *msg) {
    if (ctx) snprintf(ctx->err, sizeof(ctx->err), "%s", msg);
    return st;
}

adama_status cuda_fail(adama_ctx *ctx, const char *what, cudaError_t e) {
    if (ctx) snprintf(ctx->err, sizeof(ctx->err), "%s: %s", what, cudaGetErrorString(e));
    return ADAMA_ERR_CUDA;
}

bool aligned_to(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Makes ctx's device current for the duration of a call and restores the caller's.
struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        if (prev != dev) ok = (cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

size_t dtype_size(adama_dtype d) { return d == ADAMA_F32 ? 4 : 2; }

// ADAMA_ASYNC_COPYBACK: before `stream` may overwrite weights, it waits for the copy-back that
// is still reading them.
cudaError_t join_copyback(adama_ctx *ctx, cudaStream_t stream) {
    if (!ctx->d2h_pending) return cudaSuccess;
    ctx->d2h_pending = false;
    return cudaStreamWaitEvent(stream, ctx->ev_d2h_done, 0);
}

bool config_ok(const adama_config *cfg) {
    return cfg && cfg->beta1 >= 0.0 && cfg->beta1 < 1.0 && cfg->beta2 >= 0.0 && cfg->beta2 < 1.0 &&
           cfg->eps >= 0.0 && isfinite(cfg->eps) && cfg->device >= 0 &&
           (cfg->flags & ~(ADAMA_GRADS_PRESCALED | ADAMA_ASYNC_COPYBACK | ADAMA_INPUTS_SETTLED)) == 0;
}

adama_status check_fold_args(adama_ctx *ctx, const void *grad, adama_dtype gdt, float *m, float *v,
                             size_t n) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (gdt != ADAMA_F32 && gdt != ADAMA_BF16)
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "fold: unknown gradient dtype");
    if (n > 0 && (!grad || !m || !v)) return fail(ctx, ADAMA_ERR_INVALID_ARG, "fold: null pointer");
    if (ctx->n_micro < 1)
        return fail(ctx, ADAMA_ERR_BAD_STATE, "fold: adama_begin_minibatch has not been called");
    if (!aligned_to(grad, dtype_size(gdt)) || !aligned_to(m, 4) || !aligned_to(v, 4))
        return fail(ctx, ADAMA_ERR_MISALIGNED, "fold: pointer not aligned to its element size");
    return ADAMA_OK;
}

adama_status check_wgrad_args(adama_ctx *ctx, const void *X, const void *dY, int tokens, int d_in,
                              int d_out, int64_t ldx, int64_t ldy, float *m, float *v,
                              int64_t ldmv) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (tokens < 0 || d_in < 1 || d_out < 1)
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "wgrad_fold: bad shape");
    if (!m || !v || (tokens > 0 && (!X || !dY)))
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "wgrad_fold: null pointer");
    if (ldx < d_in || ldy < d_out || ldmv < d_out)
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "wgrad_fold: row pitch smaller than the row");
    if (ctx->n_micro < 1)
        return fail(ctx, ADAMA_ERR_BAD_STATE, "wgrad_fold: adama_begin_minibatch has not been called");
    if (!aligned_to(X, 16) || !aligned_to(dY, 16) || !aligned_to(m, 16) || !aligned_to(v, 16))
        return fail(ctx, ADAMA_ERR_MISALIGNED, "wgrad_fold: X, dY, m, v must be 16-byte aligned");
    if (ldx % 8 || ldy % 8 || ldmv % 4)
        return fail(ctx, ADAMA_ERR_MISALIGNED,
                    "wgrad_fold: ldx, ldy must be multiples of 8 and ldmv of 4");
    // tensor-map strides are limited to 2^40 bytes
    if (ldx * 2 >= (1ll << 40) || ldy * 2 >= (1ll << 40) || ldmv * 4 >= (1ll << 40))
        return fail(ctx, ADAMA_ERR_UNSUPPORTED, "wgrad_fold: row pitch too large for a tensor map");
    return ADAMA_OK;
}

adama_status check_apply_args(adama_ctx *ctx, float *w, float *m, float *v, size_t n, double lr) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (n > 0 && (!w || !m || !v)) return fail(ctx, ADAMA_ERR_INVALID_ARG, "apply: null pointer");
    if (!isfinite(lr)) return fail(ctx, ADAMA_ERR_INVALID_ARG, "apply: lr is not finite");
    if (ctx->t < 1)
        return fail(ctx, ADAMA_ERR_BAD_STATE, "apply: no mini-batch has been started (t == 0)");
    if (!aligned_to(w, 4) || !aligned_to(m, 4) || !aligned_to(v, 4))
        return fail(ctx, ADAMA_ERR_MISALIGNED, "apply: pointer not aligned to 4 bytes");
    return ADAMA_OK;
}

}  // namespace

extern "C" {

const char *adama_version(void) { return "0.1.0"; }

adama_status adama_init(adama_ctx **out, const adama_config *cfg) {
    if (!out) return ADAMA_ERR_INVALID_ARG;
    *out = nullptr;
    if (!config_ok(cfg)) return ADAMA_ERR_INVALID_ARG;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || cfg->device >= count) return ADAMA_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess) return ADAMA_ERR_CUDA;
    if (prop.major != 10) return ADAMA_ERR_UNSUPPORTED;  // kernels are built for sm_100a only

    adama_ctx *ctx = new (std::nothrow) adama_ctx();
    if (!ctx) return ADAMA_ERR_CUDA;
    memset(ctx, 0, sizeof(*ctx));
    ctx->cfg = *cfg;
    ctx->sm_count = prop.multiProcessorCount;

    DeviceGuard guard(cfg->device);
    const char *msg = "";
    cudaError_t e = guard.ok ? cudaSuccess : cudaErrorInvalidDevice;
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void **>(&ctx->status_dev), 256);
    if (e == cudaSuccess) e = cudaMemset(ctx->status_dev, 0, 256);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking);
    for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
        e = cudaEventCreateWithFlags(&ctx->ev_copied[i], cudaEventDisableTiming);
        if (e == cudaSuccess)
            e = cudaEventCreateWithFlags(&ctx->ev_folded[i], cudaEventDisableTiming);
    }
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_entry, cudaEventDisableTiming);
    if (e == cudaSuccess && (cfg->flags & ADAMA_ASYNC_COPYBACK)) {
        e = cudaStreamCreateWithFlags(&ctx->d2h_stream, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_applied, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_d2h_done, cudaEventDisableTiming);
    }
    if (e == cudaSuccess) e = adama::wgrad_fold_setup(&msg);
    if (e != cudaSuccess) {
        adama_destroy(ctx);
        return ADAMA_ERR_CUDA;
    }
    *out = ctx;
    return ADAMA_OK;
}

adama_status adama_destroy(adama_ctx *ctx) {
    if (!ctx) return ADAMA_OK;
    DeviceGuard guard(ctx->cfg.device);
    if (ctx->status_dev) cudaFree(ctx->status_dev);
    if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
    if (ctx->d2h_stream) {
        cudaStreamSynchronize(ctx->d2h_stream);  // a copy-back may still be writing host memory
        cudaStreamDestroy(ctx->d2h_stream);
    }
    if (ctx->ev_applied) cudaEventDestroy(ctx->ev_applied);
    if (ctx->ev_d2h_done) cudaEventDestroy(ctx->ev_d2h_done);
    for (int i = 0; i < 2; ++i) {
        if (ctx->ev_copied[i]) cudaEventDestroy(ctx->ev_copied[i]);
        if (ctx->ev_folded[i]) cudaEventDestroy(ctx->ev_folded[i]);
    }
    if (ctx->ev_entry) cudaEventDestroy(ctx->ev_entry);
    delete ctx;
    return ADAMA_OK;
}

adama_status adama_begin_minibatch(adama_ctx *ctx, int n_micro) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (n_micro < 1) return fail(ctx, ADAMA_ERR_INVALID_ARG, "begin_minibatch: n_micro must be >= 1");
    ctx->t += 1;
    ctx->n_micro = n_micro;
    ctx->fold_c = adama::make_fold_constants(ctx->cfg.beta1, ctx->cfg.beta2, n_micro, ctx->cfg.flags);
    return ADAMA_OK;
}

adama_status adama_fold(adama_ctx *ctx, const void *grad, adama_dtype gdt, float *m, float *v,
                        size_t n, void *cuda_stream) {
    adama_status st = check_fold_args(ctx, grad, gdt, m, v, n);
    if (st != ADAMA_OK) return st;
    if (n == 0) return ADAMA_OK;
    DeviceGuard guard(ctx->cfg.device);
    cudaError_t e = adama::launch_fold(grad, gdt, m, v, n, ctx->fold_c, ctx->sm_count,
                                       static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(ctx, "fold launch", e);
    ctx->launches += 1;
    return ADAMA_OK;
}

static adama_status wgrad_impl(adama_ctx *ctx, const void *X, const void *dY, int tokens, int d_in,
                               int d_out, int64_t ldx, int64_t ldy, float *m, float *v,
                               int64_t ldmv, float *bias_m, float *bias_v, void *cuda_stream,
                               unsigned long long wait_limit_ns = 0, int withhold_last_load = 0) {
    adama_status st = check_wgrad_args(ctx, X, dY, tokens, d_in, d_out, ldx, ldy, m, v, ldmv);
    if (st != ADAMA_OK) return st;
    if (tokens == 0) return ADAMA_OK;  // empty sum: G = 0, nothing to add
    DeviceGuard guard(ctx->cfg.device);
    adama::WgradArgs a;
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
    a.c = ctx->fold_c;
    a.status = ctx->status_dev;
    a.sm_count = ctx->sm_count;
    a.stream = static_cast<cudaStream_t>(cuda_stream);
    a.bias_m = bias_m;
    a.bias_v = bias_v;
    a.variant = ctx->variant;
    a.wait_limit_ns = wait_limit_ns;
    a.withhold_last_load = withhold_last_load;
    a.inputs_settled = (ctx->cfg.flags & ADAMA_INPUTS_SETTLED) ? 1 : 0;
    const char *msg = "wgrad_fold";
    cudaError_t e = adama::launch_wgrad_fold(a, &msg);
    if (e != cudaSuccess) return cuda_fail(ctx, msg, e);
    ctx->launches += 1;
    return ADAMA_OK;
}

adama_status adama_linear_wgrad_fold(adama_ctx *ctx, const void *X, const void *dY, int tokens,
                                     int d_in, int d_out, int64_t ldx, int64_t ldy, float *m,
                                     float *v, int64_t ldmv, void *cuda_stream) {
    return wgrad_impl(ctx, X, dY, tokens, d_in, d_out, ldx, ldy, m, v, ldmv, nullptr, nullptr,
                      cuda_stream);
}

adama_status adama_linear_wgrad_bias_fold(adama_ctx *ctx, const void *X, const void *dY, int tokens,
                                          int d_in, int d_out, int64_t ldx, int64_t ldy, float *m,
                                          float *v, int64_t ldmv, float *m_bias, float *v_bias,
                                          void *cuda_stream) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (!m_bias || !v_bias)
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "wgrad_bias_fold: null bias moments");
    if (!aligned_to(m_bias, 4) || !aligned_to(v_bias, 4))
        return fail(ctx, ADAMA_ERR_MISALIGNED, "wgrad_bias_fold: bias moments not aligned to 4 bytes");
    return wgrad_impl(ctx, X, dY, tokens, d_in, d_out, ldx, ldy, m, v, ldmv, m_bias, v_bias,
                      cuda_stream);
}

adama_status adama_linear_wgrad_fold_multi(adama_ctx *ctx, const adama_linear_item *items, int count,
                                           void *cuda_stream) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (count < 0 || (count > 0 && !items))
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "wgrad_fold_multi: null list or negative count");
    for (int i = 0; i < count; ++i) {
        const adama_linear_item &it = items[i];
        adama_status st = check_wgrad_args(ctx, it.X, it.dY, it.tokens, it.d_in, it.d_out, it.ldx,
                                           it.ldy, it.m, it.v, it.ldmv);
        if (st != ADAMA_OK) return st;
        if ((it.m_bias == nullptr) != (it.v_bias == nullptr))
            return fail(ctx, ADAMA_ERR_INVALID_ARG, "wgrad_fold_multi: m_bias and v_bias go together");
        if (!aligned_to(it.m_bias, 4) || !aligned_to(it.v_bias, 4))
            return fail(ctx, ADAMA_ERR_MISALIGNED, "wgrad_fold_multi: bias moments not aligned to 4 bytes");
    }
    DeviceGuard guard(ctx->cfg.device);
    adama::WgradArgs batch[adama::kMaxWgradLayers];
    int k = 0;
    bool first_launch = true;
    for (int i = 0; i <= count; ++i) {
        if ((i == count || k == adama::kMaxWgradLayers) && k > 0) {
            // From the call's second launch on, the kernel just before is this call's own previous
            // launch, which writes only m, v and bias moments: the operand loads need not wait for it.
            if (!first_launch) batch[0].inputs_settled = 1;
            const char *msg = "wgrad_fold_multi";
            cudaError_t e = adama::launch_wgrad_fold_multi(batch, k, &msg);
            if (e != cudaSuccess) return cuda_fail(ctx, msg, e);
            ctx->launches += 1;
            first_launch = false;
            k = 0;
        }
        if (i == count) break;
        const adama_linear_item &it = items[i];
        if (it.tokens == 0) continue;  // empty sum: nothing to add
        adama::WgradArgs &a = batch[k++];
        a = adama::WgradArgs();
        a.X = it.X;
        a.dY = it.dY;
        a.tokens = it.tokens;
        a.d_in = it.d_in;
        a.d_out = it.d_out;
        a.ldx = it.ldx;
        a.ldy = it.ldy;
        a.ldmv = it.ldmv;
        a.m = it.m;
        a.v = it.v;
        a.c = ctx->fold_c;
        a.status = ctx->status_dev;
        a.sm_count = ctx->sm_count;
        a.stream = static_cast<cudaStream_t>(cuda_stream);
        a.bias_m = it.m_bias;
        a.bias_v = it.v_bias;
        a.variant = ctx->variant;
        a.inputs_settled = (ctx->cfg.flags & ADAMA_INPUTS_SETTLED) ? 1 : 0;
    }
    return ADAMA_OK;
}

static adama_status apply_impl(adama_ctx *ctx, float *w, float *m, float *v, size_t n, double lr,
                               int world, bool sharded, void *cuda_stream,
                               void *w_bf16_out = nullptr) {
    adama_status st = check_apply_args(ctx, w, m, v, n, lr);
    if (st != ADAMA_OK) return st;
    if (world < 1) return fail(ctx, ADAMA_ERR_INVALID_ARG, "apply: world_size must be >= 1");
    if (n == 0) return ADAMA_OK;
    DeviceGuard guard(ctx->cfg.device);
    adama::ApplyConstants c = adama::make_apply_constants(ctx->cfg.beta1, ctx->cfg.beta2,
                                                          ctx->cfg.eps, ctx->t, lr, world, sharded,
                                                          ctx->weight_decay);
    cudaError_t e = join_copyback(ctx, static_cast<cudaStream_t>(cuda_stream));
    if (e == cudaSuccess)
        e = adama::launch_apply(w, m, v, n, c, ctx->sm_count,
                                static_cast<cudaStream_t>(cuda_stream), w_bf16_out);
    if (e != cudaSuccess) return cuda_fail(ctx, "apply launch", e);
    ctx->launches += 1;
    return ADAMA_OK;
}

adama_status adama_apply_bf16_copy(adama_ctx *ctx, float *w, float *m, float *v, void *w_bf16_out,
                                   size_t n, double lr, void *cuda_stream) {
    if (ctx && n > 0 && !w_bf16_out)
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "apply_bf16_copy: null bf16 output");
    if (ctx && !aligned_to(w_bf16_out, 2))
        return fail(ctx, ADAMA_ERR_MISALIGNED, "apply_bf16_copy: bf16 output not 2-byte aligned");
    return apply_impl(ctx, w, m, v, n, lr, 1, false, cuda_stream, w_bf16_out);
}

adama_status adama_apply(adama_ctx *ctx, float *w, float *m, float *v, size_t n, double lr,
                         void *cuda_stream) {
    return apply_impl(ctx, w, m, v, n, lr, 1, false, cuda_stream);
}

adama_status adama_apply_allreduced(adama_ctx *ctx, float *w, float *m, float *v, size_t n,
                                    double lr, int world_size, void *cuda_stream) {
    return apply_impl(ctx, w, m, v, n, lr, world_size, false, cuda_stream);
}

adama_status adama_apply_sharded(adama_ctx *ctx, float *w, float *m, float *v, size_t n, double lr,
                                 int world_size, void *cuda_stream) {
    return apply_impl(ctx, w, m, v, n, lr, world_size, true, cuda_stream);
}

adama_status adama_apply_sharded_peers(adama_ctx *ctx, float *const *w_peers, float *const *m_peers,
                                       float *const *v_peers, int world_size, int rank, size_t n,
                                       double lr, void *cuda_stream) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (world_size < 1 || rank < 0 || rank >= world_size || !w_peers || !m_peers || !v_peers)
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "apply_sharded_peers: bad world size, rank or list");
    if (world_size > adama::kMaxPeers)
        return fail(ctx, ADAMA_ERR_UNSUPPORTED, "apply_sharded_peers: more than 16 peers");
    if (!isfinite(lr)) return fail(ctx, ADAMA_ERR_INVALID_ARG, "apply_sharded_peers: lr is not finite");
    if (ctx->t < 1)
        return fail(ctx, ADAMA_ERR_BAD_STATE, "apply_sharded_peers: no mini-batch has been started");
    if (n % (4 * (size_t)world_size))
        return fail(ctx, ADAMA_ERR_UNSUPPORTED,
                    "apply_sharded_peers: n must be a multiple of 4*world_size (pad the buffers)");
    for (int q = 0; q < world_size; ++q) {
        if (n > 0 && (!w_peers[q] || !m_peers[q] || !v_peers[q]))
            return fail(ctx, ADAMA_ERR_INVALID_ARG, "apply_sharded_peers: null peer pointer");
        if (!aligned_to(w_peers[q], 16) || !aligned_to(m_peers[q], 16) || !aligned_to(v_peers[q], 16))
            return fail(ctx, ADAMA_ERR_MISALIGNED, "apply_sharded_peers: buffers must be 16-byte aligned");
    }
    if (n == 0) return ADAMA_OK;
    DeviceGuard guard(ctx->cfg.device);
    const adama::ApplyConstants c =
        adama::make_apply_constants(ctx->cfg.beta1, ctx->cfg.beta2, ctx->cfg.eps, ctx->t, lr,
                                    world_size, true, ctx->weight_decay);
    cudaError_t e = join_copyback(ctx, static_cast<cudaStream_t>(cuda_stream));
    if (e == cudaSuccess)
        e = adama::launch_apply_sharded_peers(w_peers, m_peers, v_peers, world_size, rank, n, c,
                                              ctx->sm_count, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(ctx, "apply_sharded_peers launch", e);
    ctx->launches += 1;
    return ADAMA_OK;
}

adama_status adama_bias_grad_fold(adama_ctx *ctx, const void *dY, int tokens, int d_out,
                                  int64_t ldy, float *m, float *v, void *cuda_stream) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (tokens < 0 || d_out < 1 || !m || !v || (tokens > 0 && !dY) || ldy < d_out)
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "bias_grad_fold: bad shape, null pointer or pitch");
    if (ctx->n_micro < 1)
        return fail(ctx, ADAMA_ERR_BAD_STATE, "bias_grad_fold: adama_begin_minibatch has not been called");
    if (!aligned_to(dY, 16) || ldy % 8 || !aligned_to(m, 4) || !aligned_to(v, 4))
        return fail(ctx, ADAMA_ERR_MISALIGNED,
                    "bias_grad_fold: dY must be 16-byte aligned with ldy a multiple of 8");
    if (tokens == 0) return ADAMA_OK;
    DeviceGuard guard(ctx->cfg.device);
    cudaError_t e = adama::launch_bias_grad_fold(dY, tokens, d_out, ldy, m, v, ctx->fold_c,
                                                 static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(ctx, "bias_grad_fold launch", e);
    ctx->launches += 1;
    return ADAMA_OK;
}

// ---- multi-tensor forms ---------------------------------------------------------------------

// Tensors at least this long go to the single-tensor kernels (they saturate the GPU alone).
static const size_t kMultiLargeThreshold = (size_t)1 << 22;

adama_status adama_fold_multi(adama_ctx *ctx, const void *const *grads, adama_dtype gdt,
                              float *const *m, float *const *v, const size_t *n, int count,
                              void *cuda_stream) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (count < 0 || (count > 0 && (!grads || !m || !v || !n)))
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "fold_multi: null list or negative count");
    for (int i = 0; i < count; ++i) {
        adama_status st = check_fold_args(ctx, grads[i], gdt, m[i], v[i], n[i]);
        if (st != ADAMA_OK) return st;
    }
    DeviceGuard guard(ctx->cfg.device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const void *g_[adama::kMultiMax];
    float *m_[adama::kMultiMax], *v_[adama::kMultiMax];
    size_t n_[adama::kMultiMax];
    int k = 0;
    cudaError_t e = cudaSuccess;
    for (int i = 0; i <= count && e == cudaSuccess; ++i) {
        const bool flush = (i == count) || k == adama::kMultiMax;
        if (flush && k > 0) {
            e = adama::launch_fold_multi(g_, gdt, m_, v_, n_, k, ctx->fold_c, ctx->sm_count, stream);
            ctx->launches += 1;
            k = 0;
        }
        if (i == count || e != cudaSuccess) break;
        if (n[i] == 0) continue;
        if (n[i] >= kMultiLargeThreshold) {
            e = adama::launch_fold(grads[i], gdt, m[i], v[i], n[i], ctx->fold_c, ctx->sm_count, stream);
            ctx->launches += 1;
            continue;
        }
        g_[k] = grads[i];
        m_[k] = m[i];
        v_[k] = v[i];
        n_[k] = n[i];
        ++k;
    }
    if (e != cudaSuccess) return cuda_fail(ctx, "fold_multi launch", e);
    return ADAMA_OK;
}

adama_status adama_apply_multi(adama_ctx *ctx, float *const *w, float *const *m, float *const *v,
                               const size_t *n, int count, double lr, void *cuda_stream) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (count < 0 || (count > 0 && (!w || !m || !v || !n)))
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "apply_multi: null list or negative count");
    for (int i = 0; i < count; ++i) {
        adama_status st = check_apply_args(ctx, w[i], m[i], v[i], n[i], lr);
        if (st != ADAMA_OK) return st;
    }
    DeviceGuard guard(ctx->cfg.device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const adama::ApplyConstants c = adama::make_apply_constants(
        ctx->cfg.beta1, ctx->cfg.beta2, ctx->cfg.eps, ctx->t, lr, 1, false, ctx->weight_decay);
    float *w_[adama::kMultiMax], *m_[adama::kMultiMax], *v_[adama::kMultiMax];
    size_t n_[adama::kMultiMax];
    int k = 0;
    cudaError_t e = join_copyback(ctx, stream);
    for (int i = 0; i <= count && e == cudaSuccess; ++i) {
        const bool flush = (i == count) || k == adama::kMultiMax;
        if (flush && k > 0) {
            e = adama::launch_apply_multi(w_, m_, v_, n_, k, c, ctx->sm_count, stream);
            ctx->launches += 1;
            k = 0;
        }
        if (i == count || e != cudaSuccess) break;
        if (n[i] == 0) continue;
        if (n[i] >= kMultiLargeThreshold) {
            e = adama::launch_apply(w[i], m[i], v[i], n[i], c, ctx->sm_count, stream);
            ctx->launches += 1;
            continue;
        }
        w_[k] = w[i];
        m_[k] = m[i];
        v_[k] = v[i];
        n_[k] = n[i];
        ++k;
    }
    if (e != cudaSuccess) return cuda_fail(ctx, "apply_multi launch", e);
    return ADAMA_OK;
}

// ---- host-buffer variants -------------------------------------------------------------------

adama_status adama_fold_host(adama_ctx *ctx, const void *grad_host, adama_dtype gdt, float *m,
                             float *v, size_t n, void *staging, size_t staging_bytes,
                             void *cuda_stream) {
    adama_status st = check_fold_args(ctx, grad_host, gdt, m, v, n);
    if (st != ADAMA_OK) return st;
    if (n == 0) return ADAMA_OK;
    if (!staging || staging_bytes < (2u << 20))
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "fold_host: staging buffer smaller than 2 MiB");
    if (!aligned_to(staging, 256))
        return fail(ctx, ADAMA_ERR_MISALIGNED, "fold_host: staging must be 256-byte aligned");
    DeviceGuard guard(ctx->cfg.device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t esz = dtype_size(gdt);
    // two halves, each a multiple of 256 bytes, so every chunk keeps m, v and grad 16-byte aligned
    const size_t half_bytes = (staging_bytes / 2) & ~(size_t)255;
    const size_t chunk = half_bytes / esz;
    char *half[2] = {static_cast<char *>(staging), static_cast<char *>(staging) + half_bytes};
    const char *src = static_cast<const char *>(grad_host);

    // the staging buffer may still be in use by earlier work on `stream`
    cudaError_t e = cudaEventRecord(ctx->ev_entry, stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_entry, 0);
    size_t done = 0;
    for (int it = 0; done < n && e == cudaSuccess; ++it) {
        const int h = it & 1;
        const size_t cnt = (n - done < chunk) ? (n - done) : chunk;
        if (it >= 2) e = cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_folded[h], 0);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(half[h], src + done * esz, cnt * esz, cudaMemcpyHostToDevice,
                                ctx->copy_stream);
        if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_copied[h], ctx->copy_stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, ctx->ev_copied[h], 0);
        if (e == cudaSuccess) {
            e = adama::launch_fold(half[h], gdt, m + done, v + done, cnt, ctx->fold_c,
                                   ctx->sm_count, stream);
            ctx->launches += 1;
        }
        if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_folded[h], stream);
        done += cnt;
    }
    if (e != cudaSuccess) return cuda_fail(ctx, "fold_host", e);
    return ADAMA_OK;
}

adama_status adama_linear_wgrad_fold_host(adama_ctx *ctx, const void *X_host, const void *dY_host,
                                          int tokens, int d_in, int d_out, float *m, float *v,
                                          int64_t ldmv, void *staging, size_t staging_bytes,
                                          void *cuda_stream) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (tokens < 0 || d_in < 1 || d_out < 1)
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "wgrad_fold_host: bad shape");
    if (d_in % 8 || d_out % 8)
        return fail(ctx, ADAMA_ERR_MISALIGNED,
                    "wgrad_fold_host: dense rows need d_in, d_out multiples of 8");
    const size_t x_bytes = (size_t)tokens * d_in * 2, y_bytes = (size_t)tokens * d_out * 2;
    const size_t y_off = (x_bytes + 255) & ~(size_t)255;
    if (!staging || staging_bytes < y_off + y_bytes)
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "wgrad_fold_host: staging buffer too small");
    if (!aligned_to(staging, 256))
        return fail(ctx, ADAMA_ERR_MISALIGNED, "wgrad_fold_host: staging must be 256-byte aligned");
    char *Xd = static_cast<char *>(staging), *Yd = Xd + y_off;
    adama_status st = check_wgrad_args(ctx, Xd, Yd, tokens, d_in, d_out, d_in, d_out, m, v, ldmv);
    if (st != ADAMA_OK) return st;
    if (tokens == 0) return ADAMA_OK;
    if (!X_host || !dY_host) return fail(ctx, ADAMA_ERR_INVALID_ARG, "wgrad_fold_host: null pointer");
    DeviceGuard guard(ctx->cfg.device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaMemcpyAsync(Xd, X_host, x_bytes, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(Yd, dY_host, y_bytes, cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) return cuda_fail(ctx, "wgrad_fold_host copy", e);
    return adama_linear_wgrad_fold(ctx, Xd, Yd, tokens, d_in, d_out, d_in, d_out, m, v, ldmv,
                                   cuda_stream);
}

adama_status adama_apply_to_host(adama_ctx *ctx, float *w, float *m, float *v, size_t n, double lr,
                                 float *w_host, void *cuda_stream) {
    if (ctx && n > 0 && !w_host)
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "apply_to_host: null host pointer");
    adama_status st = adama_apply(ctx, w, m, v, n, lr, cuda_stream);
    if (st != ADAMA_OK || n == 0) return st;
    DeviceGuard guard(ctx->cfg.device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e;
    if (ctx->cfg.flags & ADAMA_ASYNC_COPYBACK) {
        e = cudaEventRecord(ctx->ev_applied, stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->d2h_stream, ctx->ev_applied, 0);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(w_host, w, n * sizeof(float), cudaMemcpyDeviceToHost, ctx->d2h_stream);
        if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_d2h_done, ctx->d2h_stream);
        if (e == cudaSuccess) ctx->d2h_pending = true;
    } else {
        e = cudaMemcpyAsync(w_host, w, n * sizeof(float), cudaMemcpyDeviceToHost, stream);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, "apply_to_host copy", e);
    return ADAMA_OK;
}

// ---- SGD with momentum on the same pipeline; coefficient statistics ----------------------------

adama_status adama_sgdm_fold(adama_ctx *ctx, const void *grad, adama_dtype gdt, float *buf, size_t n,
                             void *cuda_stream) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (gdt != ADAMA_F32 && gdt != ADAMA_BF16)
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "sgdm_fold: unknown gradient dtype");
    if (n > 0 && (!grad || !buf)) return fail(ctx, ADAMA_ERR_INVALID_ARG, "sgdm_fold: null pointer");
    if (ctx->n_micro < 1)
        return fail(ctx, ADAMA_ERR_BAD_STATE, "sgdm_fold: adama_begin_minibatch has not been called");
    if (!aligned_to(grad, dtype_size(gdt)) || !aligned_to(buf, 4))
        return fail(ctx, ADAMA_ERR_MISALIGNED, "sgdm_fold: pointer not aligned to its element size");
    if (n == 0) return ADAMA_OK;
    DeviceGuard guard(ctx->cfg.device);
    const double N = (ctx->cfg.flags & ADAMA_GRADS_PRESCALED) ? 1.0 : (double)ctx->n_micro;
    cudaError_t e = adama::launch_sgdm_fold(grad, gdt, buf, n, (float)(1.0 / N), ctx->sm_count,
                                            static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(ctx, "sgdm_fold launch", e);
    ctx->launches += 1;
    return ADAMA_OK;
}

adama_status adama_sgdm_apply(adama_ctx *ctx, float *w, float *buf, size_t n, double lr,
                              double momentum, void *cuda_stream) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (n > 0 && (!w || !buf)) return fail(ctx, ADAMA_ERR_INVALID_ARG, "sgdm_apply: null pointer");
    if (!isfinite(lr)) return fail(ctx, ADAMA_ERR_INVALID_ARG, "sgdm_apply: lr is not finite");
    if (!(momentum >= 0.0) || !(momentum < 1.0))
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "sgdm_apply: momentum must be in [0, 1)");
    if (ctx->t < 1)
        return fail(ctx, ADAMA_ERR_BAD_STATE, "sgdm_apply: no mini-batch has been started (t == 0)");
    if (!aligned_to(w, 4) || !aligned_to(buf, 4))
        return fail(ctx, ADAMA_ERR_MISALIGNED, "sgdm_apply: pointer not aligned to 4 bytes");
    if (n == 0) return ADAMA_OK;
    DeviceGuard guard(ctx->cfg.device);
    float mu_hi, mu_lo;
    adama::split_hi_lo(momentum, &mu_hi, &mu_lo);
    cudaError_t e = join_copyback(ctx, static_cast<cudaStream_t>(cuda_stream));
    if (e == cudaSuccess)
        e = adama::launch_sgdm_apply(w, buf, n, (float)lr, mu_hi, mu_lo, ctx->sm_count,
                                     static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(ctx, "sgdm_apply launch", e);
    ctx->launches += 1;
    return ADAMA_OK;
}

adama_status adama_coefficient_stats(adama_ctx *ctx, const float *m, const float *m_begin,
                                     const float *v, float *v_adam, size_t n, double *stats_dev,
                                     void *cuda_stream) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (!stats_dev || (n > 0 && (!m || !v || !v_adam)))
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "coefficient_stats: null pointer");
    if (ctx->n_micro < 1)
        return fail(ctx, ADAMA_ERR_BAD_STATE,
                    "coefficient_stats: adama_begin_minibatch has not been called");
    if (!(ctx->cfg.beta1 < 1.0))
        return fail(ctx, ADAMA_ERR_UNSUPPORTED, "coefficient_stats: needs beta1 < 1");
    if (!aligned_to(m, 4) || !aligned_to(v, 4) || !aligned_to(v_adam, 4) ||
        (m_begin && !aligned_to(m_begin, 4)) || !aligned_to(stats_dev, 8))
        return fail(ctx, ADAMA_ERR_MISALIGNED, "coefficient_stats: pointer not aligned");
    DeviceGuard guard(ctx->cfg.device);
    adama::CoefConstants c;
    const double om1 = 1.0 - ctx->cfg.beta1;
    c.k = (float)((1.0 - ctx->cfg.beta2) / (om1 * om1));
    adama::split_hi_lo(ctx->cfg.beta2, &c.beta2_hi, &c.beta2_lo);
    cudaError_t e = adama::launch_coefficient_stats(m, m_begin, v, v_adam, n, c, stats_dev,
                                                    ctx->sm_count,
                                                    static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(ctx, "coefficient_stats launch", e);
    ctx->launches += (n > 0 ? 2 : 1);
    return ADAMA_OK;
}

// ---- state and diagnostics ------------------------------------------------------------------

int64_t adama_get_step(const adama_ctx *ctx) { return ctx ? ctx->t : -1; }

adama_status adama_set_step(adama_ctx *ctx, int64_t t) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (t < 0) return fail(ctx, ADAMA_ERR_INVALID_ARG, "set_step: t must be >= 0");
    ctx->t = t;
    return ADAMA_OK;
}

int adama_get_n_micro(const adama_ctx *ctx) { return ctx ? ctx->n_micro : -1; }

adama_status adama_set_weight_decay(adama_ctx *ctx, double weight_decay) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (!(weight_decay >= 0.0) || !isfinite(weight_decay))
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "set_weight_decay: must be finite and >= 0");
    ctx->weight_decay = weight_decay;
    return ADAMA_OK;
}

adama_status adama_sync_status(adama_ctx *ctx, void *cuda_stream) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    unsigned host[4] = {0, 0, 0, 0};
    cudaError_t e = join_copyback(ctx, stream);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(host, ctx->status_dev, sizeof(host), cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return cuda_fail(ctx, "sync_status", e);
    if (host[0] != adama::kDevOk) {
        e = cudaMemsetAsync(ctx->status_dev, 0, 256, stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
        snprintf(ctx->err, sizeof(ctx->err),
                 "device-side wait expired in the fused weight-gradient kernel "
                 "(code %u, wait %u, tile %u)",
                 host[0], host[1], host[2]);
        return ADAMA_ERR_TIMEOUT;
    }
    return ADAMA_OK;
}

adama_status adama_debug_set_status(adama_ctx *ctx, unsigned code, unsigned wait, unsigned tile,
                                    void *cuda_stream) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const unsigned words[4] = {code, wait, tile, 0};
    cudaError_t e = cudaMemcpyAsync(ctx->status_dev, words, sizeof(words), cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);  // `words` lives on this stack frame
    if (e != cudaSuccess) return cuda_fail(ctx, "debug_set_status", e);
    return ADAMA_OK;
}

adama_status adama_debug_wgrad_expire_wait(adama_ctx *ctx, const void *X, const void *dY,
                                           int tokens, int d_in, int d_out, int64_t ldx, int64_t ldy,
                                           float *m, float *v, int64_t ldmv, uint64_t wait_limit_ns,
                                           void *cuda_stream) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (wait_limit_ns < 1000 || wait_limit_ns > 1000000000ull || tokens == 0)
        return fail(ctx, ADAMA_ERR_INVALID_ARG,
                    "debug_wgrad_expire_wait: limit must be 1 us .. 1 s and tokens > 0");
    return wgrad_impl(ctx, X, dY, tokens, d_in, d_out, ldx, ldy, m, v, ldmv, nullptr, nullptr,
                      cuda_stream, wait_limit_ns, 1);
}

adama_status adama_debug_set_wgrad_variant(adama_ctx *ctx, int epilogue, int epi_warps,
                                           int box_loads, int no_pdl) {
    if (!ctx) return ADAMA_ERR_INVALID_ARG;
    if (epilogue < 0 || epilogue > 2 || (epi_warps != 0 && epi_warps != 4 && epi_warps != 8) ||
        (box_loads != 0 && box_loads != 1) || (no_pdl != 0 && no_pdl != 1))
        return fail(ctx, ADAMA_ERR_INVALID_ARG, "debug_set_wgrad_variant: value out of range");
    ctx->variant.epilogue = epilogue;
    ctx->variant.epi_warps = epi_warps;
    ctx->variant.box_loads = box_loads;
    ctx->variant.no_pdl = no_pdl;
    return ADAMA_OK;
}

int adama_debug_setup_state(int device) { return adama::wgrad_setup_state(device); }

const char *adama_last_error(const adama_ctx *ctx) { return ctx ? ctx->err : ""; }

int64_t adama_launch_count(const adama_ctx *ctx) { return ctx ? ctx->launches : -1; }

adama_status adama_host_constants(const adama_config *cfg, int n_micro, int64_t t, double lr,
                                  float out[9]) {
    return adama_host_constants_allreduced(cfg, n_micro, t, lr, 1, out);
}

adama_status adama_host_constants_sharded(const adama_config *cfg, int n_micro, int64_t t, double lr,
                                          int world_size, float out[9]) {
    adama_status st = adama_host_constants_allreduced(cfg, n_micro, t, lr, world_size, out);
    if (st != ADAMA_OK) return st;
    adama::ApplyConstants c =
        adama::make_apply_constants(cfg->beta1, cfg->beta2, cfg->eps, t, lr, world_size, true);
    out[5] = c.beta1_hi;
    out[6] = c.beta1_lo;
    out[7] = c.beta2_hi;
    out[8] = c.beta2_lo;
    return ADAMA_OK;
}

adama_status adama_host_constants_allreduced(const adama_config *cfg, int n_micro, int64_t t,
                                             double lr, int world_size, float out[9]) {
    if (!config_ok(cfg) || !out || n_micro < 1 || t < 1 || world_size < 1)
        return ADAMA_ERR_INVALID_ARG;
    adama::FoldConstants f = adama::make_fold_constants(cfg->beta1, cfg->beta2, n_micro, cfg->flags);
    adama::ApplyConstants c =
        adama::make_apply_constants(cfg->beta1, cfg->beta2, cfg->eps, t, lr, world_size);
    out[0] = f.a;
    out[1] = f.b;
    out[2] = c.step;
    out[3] = c.inv_bc2;
    out[4] = c.eps;
    out[5] = c.beta1_hi;
    out[6] = c.beta1_lo;
    out[7] = c.beta2_hi;
    out[8] = c.beta2_lo;
    return ADAMA_OK;
}

}  // extern "C"
