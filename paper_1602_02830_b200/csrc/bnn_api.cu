// Context management, status strings and the host-side BatchNorm fold.
#include "bnn_common.cuh"
#include <cmath>
#include <new>

extern "C" int bnn_create(bnn_ctx **out, int device, void *cuda_stream) {
    if (!out) return BNN_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return BNN_ERR_CUDA;
    bnn_ctx *c = new (std::nothrow) bnn_ctx();
    if (!c) return BNN_ERR_INVALID_ARG;
    c->device = device;
    c->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    c->ws = nullptr;
    c->ws_bytes = 0;
    c->last_cuda_error = 0;
    c->sm_count = 0;
    c->variant = 0;
    c->engine = 0;
    c->tile_rows = 8;
    c->pair_mode = 0;
    c->operand_bits = 4;
    c->wait_limit_ns = 2000000000ull;
    c->drop_loads = 0;
    c->conv_form = 0;
    c->filter_repetition = 0;
    c->last_kernel[0] = 0;
    c->copy_stream = nullptr;
    c->copy_ready = false;
    for (int i = 0; i < 8; ++i) c->ev[i] = nullptr;
    if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
        delete c;
        return BNN_ERR_CUDA;
    }
    *out = c;
    return BNN_OK;
}

extern "C" int bnn_destroy(bnn_ctx *ctx) {
    if (!ctx) return BNN_ERR_INVALID_ARG;
    if (ctx->copy_ready) {
        bnn_device_guard guard(ctx);
        if (guard.ok) {
            cudaStreamSynchronize(ctx->copy_stream);
            for (int i = 0; i < 8; ++i) cudaEventDestroy(ctx->ev[i]);
            cudaStreamDestroy(ctx->copy_stream);
        }
    }
    delete ctx;
    return BNN_OK;
}

extern "C" const char *bnn_status_string(int status) {
    switch (status) {
        case BNN_OK: return "ok";
        case BNN_ERR_INVALID_ARG: return "invalid argument";
        case BNN_ERR_ALIGNMENT: return "pointer or leading dimension not aligned as required";
        case BNN_ERR_WORKSPACE: return "workspace missing or too small";
        case BNN_ERR_CUDA: return "CUDA runtime error";
        case BNN_ERR_DEVICE_STATUS: return "kernel reported an internal error";
        case BNN_ERR_TOO_LARGE: return "problem exceeds the built-in scratch of the no-allocation entry point";
        default: return "unknown status";
    }
}

extern "C" int bnn_set_popc_variant(bnn_ctx *ctx, int variant) {
    if (!ctx || variant < 0 || variant > 2) return BNN_ERR_INVALID_ARG;
    ctx->variant = variant;
    return BNN_OK;
}

extern "C" int bnn_set_tile_rows(bnn_ctx *ctx, int rows) {
    if (!ctx || (rows != 8 && rows != 16)) return BNN_ERR_INVALID_ARG;
    ctx->tile_rows = rows;
    return BNN_OK;
}

extern "C" int bnn_set_pair_mode(bnn_ctx *ctx, int mode) {
    if (!ctx || mode < 0 || mode > 2) return BNN_ERR_INVALID_ARG;
    ctx->pair_mode = mode;
    return BNN_OK;
}

extern "C" int bnn_set_operand_bits(bnn_ctx *ctx, int bits) {
    if (!ctx || (bits != 4 && bits != 8)) return BNN_ERR_INVALID_ARG;
    ctx->operand_bits = bits;
    return BNN_OK;
}

extern "C" int bnn_set_wait_limit_ns(bnn_ctx *ctx, uint64_t ns) {
    if (!ctx || ns == 0 || ns > 60000000000ull) return BNN_ERR_INVALID_ARG;
    ctx->wait_limit_ns = ns;
    return BNN_OK;
}

extern "C" int bnn_set_conv_filter_repetition(bnn_ctx *ctx, int on) {
    if (!ctx || (on != 0 && on != 1)) return BNN_ERR_INVALID_ARG;
    ctx->filter_repetition = on;
    return BNN_OK;
}

extern "C" int bnn_set_conv_form(bnn_ctx *ctx, int form) {
    if (!ctx || (form != 0 && form != 1)) return BNN_ERR_INVALID_ARG;
    ctx->conv_form = form;
    return BNN_OK;
}

extern "C" int bnn_debug_drop_loads(bnn_ctx *ctx, int on) {
    if (!ctx || (on != 0 && on != 1)) return BNN_ERR_INVALID_ARG;
    ctx->drop_loads = on;
    return BNN_OK;
}

extern "C" int bnn_set_engine(bnn_ctx *ctx, int engine) {
    if (!ctx || engine < 0 || engine > 2) return BNN_ERR_INVALID_ARG;
    ctx->engine = engine;
    return BNN_OK;
}

extern "C" const char *bnn_last_tensor_kernel(const bnn_ctx *ctx) { return ctx ? ctx->last_kernel : ""; }

extern "C" int bnn_last_cuda_error(const bnn_ctx *ctx) { return ctx ? ctx->last_cuda_error : 0; }

extern "C" int bnn_set_workspace(bnn_ctx *ctx, void *dptr, size_t bytes) {
    if (!ctx) return BNN_ERR_INVALID_ARG;
    if ((dptr == nullptr) != (bytes == 0)) return BNN_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(dptr) & 255u) return BNN_ERR_ALIGNMENT;
    ctx->ws = dptr;
    ctx->ws_bytes = bytes;
    return BNN_OK;
}

// Run-time BatchNorm of an integer pre-activation in double (Algorithm 4: BatchNorm(a_k, theta_k)),
// operations in this order: subtract, divide by the root, scale, shift.  This translation unit is
// compiled without floating-point contraction so that each operation rounds on its own.
static inline double bn_eval(double x, double g, double b, double mu, double var, double eps) {
    const double xhat = (x - mu) / std::sqrt(var + eps);
    return g * xhat + b;
}

// Sign(BN(x)) is a monotone step in x (every operation above is monotone in x for a fixed sign of
// gamma), so one integer threshold reproduces it exactly; it is located by bisection on the
// double-precision BatchNorm itself rather than by solving for the crossing in closed form.
extern "C" int bnn_fold_batchnorm(const float *gamma, const float *beta, const float *mean, const float *var,
                                  double eps, int64_t n, int64_t x_max, int32_t *thr, uint32_t *flip) {
    if (n < 0 || x_max < 0 || x_max > 0x3fffffff) return BNN_ERR_INVALID_ARG;
    if (n == 0) return BNN_OK;
    if (!gamma || !beta || !mean || !var || !thr || !flip) return BNN_ERR_INVALID_ARG;
    for (int64_t w = 0; w < (n + 31) / 32; ++w) flip[w] = 0u;
    for (int64_t c = 0; c < n; ++c) {
        const double g = gamma[c], b = beta[c], mu = mean[c], v = var[c];
        if (!(v + eps > 0.0) || std::isnan(g) || std::isnan(b) || std::isnan(mu)) return BNN_ERR_INVALID_ARG;
        auto plus = [&](int64_t x) { return bn_eval((double)x, g, b, mu, v, eps) >= 0.0; };
        int32_t t;
        bool f;
        if (g == 0.0) {                       // constant output Sign(beta)
            t = (int32_t)(-x_max);
            f = !plus(0);
        } else if (g > 0.0) {                 // +1 for x >= t : smallest x in [-x_max, x_max+1] that is plus
            int64_t lo = -x_max, hi = x_max + 1;          // invariant: everything >= hi is plus (or hi is the sentinel)
            while (lo < hi) {
                const int64_t mid = lo + (hi - lo) / 2;   // mid <= x_max
                if (plus(mid)) hi = mid; else lo = mid + 1;
            }
            t = (int32_t)lo;
            f = false;
        } else {                              // +1 for x <= u : bit = (x >= u+1) XOR 1
            int64_t lo = -x_max, hi = x_max + 1;          // smallest x that is NOT plus
            while (lo < hi) {
                const int64_t mid = lo + (hi - lo) / 2;
                if (!plus(mid)) hi = mid; else lo = mid + 1;
            }
            t = (int32_t)lo;
            f = true;
        }
        thr[c] = t;
        if (f) flip[c / 32] |= (1u << (c % 32));
    }
    return BNN_OK;
}
