// bnn_mlp_forward: Algorithm 4 ("Running a BNN") as a sequence of stream-ordered launches:
// bit-plane first layer -> fused binary dense layers -> real-valued output layer.
#include "bnn_internal.cuh"
#include <mutex>

namespace {

inline int64_t act_ld(int64_t n) { return ((n + 127) / 128) * 4; }   // packed leading dimension, multiple of 4 words
inline size_t round256(size_t b) { return (b + 255) & ~size_t(255); }

int check_desc(const bnn_mlp_desc *m) {
    if (!m || m->n_layers < 2 || !m->layers) return BNN_ERR_INVALID_ARG;
    for (int k = 0; k < m->n_layers; ++k) {
        const bnn_layer_desc &L = m->layers[k];
        if (L.K <= 0 || L.N <= 0 || !L.Wp) return BNN_ERR_INVALID_ARG;
        if (int st = bnn_check_packed(L.Wp, L.ldw_w, L.K, L.N)) return st;   // every kernel reads the rows with 128-bit loads
        if ((L.W8 && !bnn_aligned16(L.W8)) || (L.W4 && !bnn_aligned16(L.W4))) return BNN_ERR_ALIGNMENT;
        if (k > 0 && L.K != m->layers[k - 1].N) return BNN_ERR_INVALID_ARG;
        if (k < m->n_layers - 1) {
            if (!L.thr) return BNN_ERR_INVALID_ARG;
        } else {
            if (!L.gamma || !L.beta || !L.mean || !L.var) return BNN_ERR_INVALID_ARG;
            if (L.N > 32) return BNN_ERR_INVALID_ARG;   // output layer runs on the skinny kernel
        }
    }
    return BNN_OK;
}

size_t act_bytes(const bnn_mlp_desc *m, int64_t batch) {
    int64_t widest = 0;
    for (int k = 0; k < m->n_layers - 1; ++k) widest = m->layers[k].N > widest ? m->layers[k].N : widest;
    return round256((size_t)batch * act_ld(widest) * 4);
}

// Hides the context's workspace for the duration of a call and puts it back on scope exit.
struct workspace_hide {
    bnn_ctx *ctx;
    void *ws;
    size_t bytes;
    explicit workspace_hide(bnn_ctx *c) : ctx(c), ws(c->ws), bytes(c->ws_bytes) { c->ws = nullptr; c->ws_bytes = 0; }
    ~workspace_hide() { ctx->ws = ws; ctx->ws_bytes = bytes; }
};

// Restores the context's engine choice on scope exit.
struct engine_pin {
    bnn_ctx *ctx;
    int saved;
    engine_pin(bnn_ctx *c, int engine) : ctx(c), saved(c->engine) { c->engine = engine; }
    ~engine_pin() { ctx->engine = saved; }
};

int forward_device(bnn_ctx *ctx, const bnn_mlp_desc *m, const uint8_t *X, int64_t ldx, int64_t batch, float *scores,
                   int64_t lds, uint32_t *const *hidden_out, char *ws, void *planes_scratch = nullptr) {
    // The layer calls below must stay on the CUDA-core kernels: the tensor engine would expand operands into the
    // context's workspace, which may be the very memory `ws` points into.
    engine_pin pin(ctx, BNN_ENGINE_POPC);
    const size_t ab = act_bytes(m, batch);
    uint32_t *bufs[2] = {reinterpret_cast<uint32_t *>(ws), reinterpret_cast<uint32_t *>(ws + ab)};
    const int L = m->n_layers;
    const uint32_t *cur = nullptr;
    for (int k = 0; k < L - 1; ++k) {
        const bnn_layer_desc &D = m->layers[k];
        uint32_t *dst = bufs[k & 1];
        const int64_t ldo = act_ld(D.N);
        int st;
        if (k == 0 && planes_scratch && D.N >= 512)
            st = bnn_first_layer_planes_pre(ctx, X, ldx, D.Wp, D.ldw_w, D.thr, D.flip, dst, ldo, nullptr, 0, batch, D.N, D.K,
                                            planes_scratch);
        else if (k == 0)
            st = bnn_first_layer_bitplanes(ctx, X, ldx, D.Wp, D.ldw_w, D.thr, D.flip, dst, ldo, nullptr, 0, batch, D.N, D.K);
        else
            st = bnn_binary_dense(ctx, cur, act_ld(D.K), D.Wp, D.ldw_w, D.thr, D.flip, dst, ldo, batch, D.N, D.K);
        if (st) return st;
        if (hidden_out && hidden_out[k])
            BNN_CUDA_TRY(ctx, cudaMemcpyAsync(hidden_out[k], dst, (size_t)batch * ldo * 4, cudaMemcpyDeviceToDevice,
                                              ctx->stream));
        cur = dst;
    }
    const bnn_layer_desc &O = m->layers[L - 1];
    return bnn_output_scores(ctx, cur, act_ld(O.K), O.Wp, O.ldw_w, O.gamma, O.beta, O.mean, O.var, O.eps, scores, lds,
                             batch, O.N, O.K);
}

// Bytes the tensor-core engine adds: two byte-per-value activation buffers and one expanded weight matrix.
size_t tensor_act8_bytes(const bnn_mlp_desc *m, int64_t batch) {
    int64_t widest = 0;
    for (int k = 0; k < m->n_layers - 1; ++k) widest = m->layers[k].N > widest ? m->layers[k].N : widest;
    return bnn_umma_operand_bytes(batch, widest);
}
size_t tensor_w8_bytes(const bnn_mlp_desc *m) {
    size_t w = 0;
    for (int k = 0; k < m->n_layers - 1; ++k) {
        const size_t b = bnn_umma_operand_bytes(m->layers[k].N, m->layers[k].K);
        w = b > w ? b : w;
    }
    return w;
}
bool tensor_applies(const bnn_ctx *ctx, const bnn_mlp_desc *m, int64_t batch) {
    if (ctx->engine == BNN_ENGINE_POPC) return false;
    for (int k = 0; k < m->n_layers - 1; ++k)
        if (!bnn_umma_shape_ok(batch, m->layers[k].N, m->layers[k].K)) return false;
    return true;
}

// The same layer sequence on the tensor-core engine.  Every hidden layer writes its signs twice: packed (the
// ABI's activation format, read by the output layer and by hidden_out) and as +-1 bytes (next layer's operand).
int forward_device_tensor(bnn_ctx *ctx, const bnn_mlp_desc *m, const uint8_t *X, int64_t ldx, int64_t batch, float *scores,
                          int64_t lds, uint32_t *const *hidden_out, char *ws) {
    const size_t ab = act_bytes(m, batch), a8 = tensor_act8_bytes(m, batch);
    uint32_t *bits[2] = {reinterpret_cast<uint32_t *>(ws), reinterpret_cast<uint32_t *>(ws + ab)};
    int8_t *act8[2] = {reinterpret_cast<int8_t *>(ws + 2 * ab), reinterpret_cast<int8_t *>(ws + 2 * ab + a8)};
    int8_t *W8 = reinterpret_cast<int8_t *>(ws + 2 * ab + 2 * a8);
    const int L = m->n_layers;
    // +-1 activations travel between hidden layers as e2m1 nibbles (4-bit engine) or as signed bytes
    const bool f4 = ctx->operand_bits == 4;
    const uint32_t *cur = nullptr;
    const int8_t *cur8 = nullptr;
    for (int k = 0; k < L - 1; ++k) {
        const bnn_layer_desc &D = m->layers[k];
        uint32_t *dst = bits[k & 1];
        int8_t *dst8 = act8[k & 1];
        const int64_t ldo = act_ld(D.N);
        const bool need_next = (k < L - 2);
        // packed sign words are only needed by the output layer and by callers who asked for the hidden activations;
        // the next hidden layer reads the expanded operand
        uint32_t *dst_bits = (!need_next || (hidden_out && hidden_out[k])) ? dst : nullptr;
        const int64_t ld_next = f4 ? bnn_umma_operand_ld_f4(D.N) : bnn_umma_operand_ld(D.N);
        int st;
        if (k == 0 || !f4) {
            const int8_t *Wk8 = D.W8;                  // expanded once by the caller, or here on every call
            if (!Wk8) {
                if ((st = bnn_umma_expand(ctx, D.Wp, D.ldw_w, D.N, D.K, W8))) return st;
                Wk8 = W8;
            }
            st = bnn_umma_gemm(ctx, k == 0 ? static_cast<const void *>(X) : cur8, k == 0 ? ldx : bnn_umma_operand_ld(D.K), k == 0, Wk8,
                               bnn_umma_operand_ld(D.K), batch, D.N, D.K, nullptr, 0, D.thr, D.flip, dst_bits, ldo,
                               need_next ? dst8 : nullptr, ld_next, 0, 0, 0, f4 ? 1 : 0,
                               (k > 0 && D.W8) ? 1 : 0);   // from layer 2 on the kernel before wrote activations, not these weights
        } else {
            const uint8_t *Wk4 = D.W4;
            if (!Wk4) {
                if ((st = bnn_umma_expand_f4(ctx, D.Wp, D.ldw_w, D.N, D.K, reinterpret_cast<uint8_t *>(W8)))) return st;
                Wk4 = reinterpret_cast<uint8_t *>(W8);
            }
            st = bnn_umma_gemm_f4(ctx, reinterpret_cast<const uint8_t *>(cur8), bnn_umma_operand_ld_f4(D.K), Wk4,
                                  bnn_umma_operand_ld_f4(D.K), batch, D.N, D.K, nullptr, 0, D.thr, D.flip, dst_bits, ldo,
                                  need_next ? reinterpret_cast<uint8_t *>(dst8) : nullptr, ld_next, D.W4 ? 1 : 0);
        }
        if (st) return st;
        if (hidden_out && hidden_out[k])
            BNN_CUDA_TRY(ctx, cudaMemcpyAsync(hidden_out[k], dst, (size_t)batch * ldo * 4, cudaMemcpyDeviceToDevice,
                                              ctx->stream));
        cur = dst;
        cur8 = dst8;
    }
    const bnn_layer_desc &O = m->layers[L - 1];
    return bnn_output_scores(ctx, cur, act_ld(O.K), O.Wp, O.ldw_w, O.gamma, O.beta, O.mean, O.var, O.eps, scores, lds,
                             batch, O.N, O.K);
}

size_t tensor_extra_bytes(const bnn_mlp_desc *m, int64_t batch) {
    return 2 * tensor_act8_bytes(m, batch) + tensor_w8_bytes(m);
}

}  // namespace

// Offset of the bit-plane scratch of the CUDA-core first layer inside the workspace: behind the activation buffers
// and (when the shapes qualify) the tensor engine's buffers.
static size_t planes_offset(const bnn_mlp_desc *m, int64_t batch) {
    size_t b = 2 * act_bytes(m, batch);
    bool all = true;
    for (int k = 0; k < m->n_layers - 1; ++k)
        if (!bnn_umma_shape_ok(batch, m->layers[k].N, m->layers[k].K)) all = false;
    if (all) b += tensor_extra_bytes(m, batch);      // room for the tensor-core engine, whatever engine is selected later
    return b;
}

extern "C" size_t bnn_mlp_workspace_bytes(const bnn_mlp_desc *m, int64_t batch, int host_io) {
    if (check_desc(m) != BNN_OK || batch <= 0) return 0;
    size_t b = planes_offset(m, batch) + bnn_planes_scratch_bytes(batch, m->layers[0].K);
    if (host_io) {
        b += round256((size_t)batch * m->layers[0].K);                        // staged input
        b += round256((size_t)batch * m->layers[m->n_layers - 1].N * 4);      // staged scores
    }
    return b;
}

extern "C" int bnn_mlp_forward(bnn_ctx *ctx, const bnn_mlp_desc *m, const uint8_t *X, int64_t ldx, int64_t batch,
                               float *scores, int64_t lds, uint32_t *const *hidden_out) {
    if (int st = check_desc(m)) return st;      // the descriptor first: its errors need no context to be found
    if (!ctx || batch < 0) return BNN_ERR_INVALID_ARG;
    if (batch == 0) return BNN_OK;
    if (!X || !scores || ldx < m->layers[0].K || lds < m->layers[m->n_layers - 1].N) return BNN_ERR_INVALID_ARG;
    if (!ctx->ws || ctx->ws_bytes < bnn_mlp_workspace_bytes(m, batch, 0)) return BNN_ERR_WORKSPACE;
    bnn_device_guard guard(ctx);
    if (!guard.ok) return BNN_ERR_CUDA;
    if (tensor_applies(ctx, m, batch) && (ldx % 16) == 0 && bnn_aligned16(X))
        return forward_device_tensor(ctx, m, X, ldx, batch, scores, lds, hidden_out, static_cast<char *>(ctx->ws));
    return forward_device(ctx, m, X, ldx, batch, scores, lds, hidden_out, static_cast<char *>(ctx->ws),
                          static_cast<char *>(ctx->ws) + planes_offset(m, batch));
}

extern "C" int bnn_mlp_forward_host(bnn_ctx *ctx, const bnn_mlp_desc *m, const uint8_t *X_host, int64_t ldx,
                                    int64_t batch, float *scores_host, int64_t lds) {
    if (int st = check_desc(m)) return st;      // the descriptor first: its errors need no context to be found
    if (!ctx || batch < 0) return BNN_ERR_INVALID_ARG;
    if (batch == 0) return BNN_OK;
    const int64_t K0 = m->layers[0].K, NL = m->layers[m->n_layers - 1].N;
    if (!X_host || !scores_host || ldx < K0 || lds < NL) return BNN_ERR_INVALID_ARG;
    if (!ctx->ws || ctx->ws_bytes < bnn_mlp_workspace_bytes(m, batch, 1)) return BNN_ERR_WORKSPACE;
    bnn_device_guard guard(ctx);
    if (!guard.ok) return BNN_ERR_CUDA;
    char *ws = static_cast<char *>(ctx->ws);
    const bool tensor = tensor_applies(ctx, m, batch) && (K0 % 16) == 0;
    // staging buffers sit behind everything the device-side forward may use
    const size_t fwd = bnn_mlp_workspace_bytes(m, batch, 0);
    uint8_t *Xd = reinterpret_cast<uint8_t *>(ws + fwd);
    float *Sd = reinterpret_cast<float *>(ws + fwd + round256((size_t)batch * K0));

    // Row chunks are independent through every layer, so for a large batch on the tensor engine the input is copied
    // in chunks on an internal stream while the previous chunk is already running through the layers.  Every chunk
    // pays the fixed cost of its four kernels, so there are only two, the first the smaller one (its copy is not
    // overlapped with anything): boundaries at multiples of 128 rows (whole tiles).
#ifndef BNN_E2E_SPLIT_PCT
#define BNN_E2E_SPLIT_PCT 40
#endif
#ifndef BNN_E2E_SPLIT2_PCT
#define BNN_E2E_SPLIT2_PCT 0          // second boundary (0: two chunks)
#endif
    int nchunks = 1;
    int64_t bounds[5] = {0, batch, batch, batch, batch};
    if (tensor && batch >= 6144) {
        const int64_t first = ((batch * BNN_E2E_SPLIT_PCT / 100 + 127) / 128) * 128;
        const int64_t second = ((batch * BNN_E2E_SPLIT2_PCT / 100 + 127) / 128) * 128;
        if (first > 0 && first < batch && tensor_applies(ctx, m, first) && tensor_applies(ctx, m, batch - first)) {
            nchunks = 2;
            bounds[1] = first;
            if (BNN_E2E_SPLIT2_PCT > 0 && second > first && second < batch && tensor_applies(ctx, m, second - first) &&
                tensor_applies(ctx, m, batch - second)) {
                nchunks = 3;
                bounds[2] = second;
            }
        }
    }
    if (nchunks > 1 && !ctx->copy_ready) {
        BNN_CUDA_TRY(ctx, cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
        for (int i = 0; i < 8; ++i) BNN_CUDA_TRY(ctx, cudaEventCreateWithFlags(&ctx->ev[i], cudaEventDisableTiming));
        ctx->copy_ready = true;
    }
    cudaStream_t cs = nchunks > 1 ? ctx->copy_stream : ctx->stream;
    if (nchunks > 1) {   // the copies may not overtake work that is already queued on the context's stream
        BNN_CUDA_TRY(ctx, cudaEventRecord(ctx->ev[0], ctx->stream));
        BNN_CUDA_TRY(ctx, cudaStreamWaitEvent(cs, ctx->ev[0], 0));
    }
    for (int c = 0; c < nchunks; ++c) {
        const int64_t r0 = bounds[c], rows = bounds[c + 1] - r0;
        if (ldx == K0)   // contiguous: one linear copy
            BNN_CUDA_TRY(ctx, cudaMemcpyAsync(Xd + r0 * K0, X_host + r0 * ldx, (size_t)K0 * rows, cudaMemcpyHostToDevice, cs));
        else
            BNN_CUDA_TRY(ctx, cudaMemcpy2DAsync(Xd + r0 * K0, (size_t)K0, X_host + r0 * ldx, (size_t)ldx, (size_t)K0, (size_t)rows,
                                                cudaMemcpyHostToDevice, cs));
        if (nchunks > 1) BNN_CUDA_TRY(ctx, cudaEventRecord(ctx->ev[1 + c], cs));
    }
    for (int c = 0; c < nchunks; ++c) {
        const int64_t r0 = bounds[c], rows = bounds[c + 1] - r0;
        if (nchunks > 1) BNN_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->stream, ctx->ev[1 + c], 0));
        if (int st = tensor ? forward_device_tensor(ctx, m, Xd + r0 * K0, K0, rows, Sd + r0 * NL, NL, nullptr, ws)
                            : forward_device(ctx, m, Xd + r0 * K0, K0, rows, Sd + r0 * NL, NL, nullptr, ws,
                                             ws + planes_offset(m, batch)))
            return st;
        if (nchunks > 1 && c + 1 < nchunks) {
            // this chunk's scores travel back on the copy stream while the next chunk runs through the layers
            BNN_CUDA_TRY(ctx, cudaEventRecord(ctx->ev[5], ctx->stream));
            BNN_CUDA_TRY(ctx, cudaStreamWaitEvent(cs, ctx->ev[5], 0));
            if (lds == NL)
                BNN_CUDA_TRY(ctx, cudaMemcpyAsync(scores_host + r0 * lds, Sd + r0 * NL, (size_t)NL * 4 * rows, cudaMemcpyDeviceToHost, cs));
            else
                BNN_CUDA_TRY(ctx, cudaMemcpy2DAsync(scores_host + r0 * lds, (size_t)lds * 4, Sd + r0 * NL, (size_t)NL * 4,
                                                    (size_t)NL * 4, (size_t)rows, cudaMemcpyDeviceToHost, cs));
            BNN_CUDA_TRY(ctx, cudaEventRecord(ctx->ev[6], cs));
        }
    }
    {
        // the last chunk's (or all) scores on the context's stream, which also waits for the earlier chunks' copies
        const int64_t r0 = bounds[nchunks - 1], rows = batch - r0;
        if (lds == NL)
            BNN_CUDA_TRY(ctx, cudaMemcpyAsync(scores_host + r0 * lds, Sd + r0 * NL, (size_t)NL * 4 * rows, cudaMemcpyDeviceToHost,
                                              ctx->stream));
        else
            BNN_CUDA_TRY(ctx, cudaMemcpy2DAsync(scores_host + r0 * lds, (size_t)lds * 4, Sd + r0 * NL, (size_t)NL * 4, (size_t)NL * 4,
                                                (size_t)rows, cudaMemcpyDeviceToHost, ctx->stream));
        if (nchunks > 1) BNN_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->stream, ctx->ev[6], 0));
    }
    return BNN_OK;
}

// ---------------------------------------------------------------------------------------------------
// bnn_mlp_forward_noalloc: the same forward pass for callers that must not allocate device memory.
//
// The two activation buffers that bnn_mlp_forward takes from the caller's workspace live here in a
// file-scope device array instead.  It is part of the library image: every GPU that loads the library
// holds these bytes until the process exits, which is why the limit is kept modest.
//
// In host code the array's name is only a host-side stand-in for the symbol, not a device address, so the
// address is obtained once per device with cudaGetSymbolAddress (with that device current) and that
// pointer is what the kernels receive.
namespace {

constexpr size_t kNoAllocBufferBytes = 512u * 1024u;   // per activation buffer; two buffers
constexpr int kNoAllocMaxDevices = 64;

static __device__ __align__(256) unsigned char g_noalloc_scratch[2 * kNoAllocBufferBytes];

std::mutex g_noalloc_mutex;
void *g_noalloc_ptr[kNoAllocMaxDevices] = {};

// Device address of the scratch array on ctx's device (which the caller has made current).
int noalloc_scratch(bnn_ctx *ctx, char **out) {
    if (ctx->device < 0 || ctx->device >= kNoAllocMaxDevices) return BNN_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[ctx->device]) {
        void *ptr = nullptr;
        BNN_CUDA_TRY(ctx, cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
        if (!ptr) return BNN_ERR_CUDA;
        g_noalloc_ptr[ctx->device] = ptr;
    }
    *out = static_cast<char *>(g_noalloc_ptr[ctx->device]);
    return BNN_OK;
}

}  // namespace

extern "C" size_t bnn_mlp_noalloc_max_bytes(void) { return kNoAllocBufferBytes; }

extern "C" int bnn_mlp_forward_noalloc(bnn_ctx *ctx, const bnn_mlp_desc *m, const uint8_t *X, int64_t ldx,
                                       int64_t batch, float *scores, int64_t lds) {
    if (int st = check_desc(m)) return st;      // the descriptor first: its errors need no context to be found
    if (!ctx || batch < 0) return BNN_ERR_INVALID_ARG;
    if (batch == 0) return BNN_OK;
    if (!X || !scores || ldx < m->layers[0].K || lds < m->layers[m->n_layers - 1].N) return BNN_ERR_INVALID_ARG;
    // one activation buffer = batch rows of the widest hidden layer, packed; it must fit the built-in array
    if (act_bytes(m, batch) > kNoAllocBufferBytes) return BNN_ERR_TOO_LARGE;
    bnn_device_guard guard(ctx);
    if (!guard.ok) return BNN_ERR_CUDA;
    char *scratch = nullptr;
    if (int st = noalloc_scratch(ctx, &scratch)) return st;
    // Nothing in the scratch has to start at zero: every layer writes all words of its output rows, padding
    // included, before the next layer reads them; what an earlier call left behind is never read.
    // A workspace that the caller lent to the context for other calls stays untouched: with it hidden, the first layer
    // takes its fused form, which needs no bit-plane scratch, and no layer can pick the tensor engine.
    workspace_hide hide(ctx);
    return forward_device(ctx, m, X, ldx, batch, scores, lds, nullptr, scratch);
}
