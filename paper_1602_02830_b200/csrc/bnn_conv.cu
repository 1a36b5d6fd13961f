// bnn_binary_conv2d: 3x3 / pad 1 binary convolution as an implicit GEMM over the tiled kernel, and the
// 8-bit first convolution by bit-planes (Section 3.3; Section 1.6 for the first layer).
#include "bnn_internal.cuh"

using namespace bnn_tile;

namespace {

// First convolution: 9 * C_in <= 32, so the whole receptive field of a pixel is one word per bit-plane.
// s = sum_p 2^p * (2 * popc(x^p & w_plus) - popc(x^p)) = 2 * sum_p 2^p popc(x^p & w_plus) - sum(x);
// taps outside the image hold x = 0 and drop out by themselves.
// One thread per output pixel (per pooling window when pooling), loop over the filters held in shared memory.
struct ConvU8Args {
    const uint8_t *act; int64_t B; int H, W, Cin;
    const uint32_t *Wp; int64_t Cout;
    int pool;
    const int32_t *thr; const uint32_t *flip;
    uint32_t *out_bits; int32_t *out_sums;
};

__global__ void __launch_bounds__(128) k_conv_u8_planes(const ConvU8Args p) {
    extern __shared__ uint32_t wsm[];   // Cout filter words
    for (int64_t e = threadIdx.x; e < p.Cout; e += blockDim.x) wsm[e] = p.Wp[e];
    __syncthreads();
    const int Ho = p.pool ? p.H / 2 : p.H, Wo = p.pool ? p.W / 2 : p.W;
    const int64_t total = p.B * Ho * Wo;
    const int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (o >= total) return;
    const int xo = (int)(o % Wo), yo = (int)((o / Wo) % Ho);
    const int64_t b = o / ((int64_t)Wo * Ho);
    const int npix = p.pool ? 4 : 1;
    uint32_t planes[4][8];
    int32_t xsum[4];
    for (int q = 0; q < npix; ++q) {
        const int y = p.pool ? 2 * yo + (q >> 1) : yo, x = p.pool ? 2 * xo + (q & 1) : xo;
#pragma unroll
        for (int pl = 0; pl < 8; ++pl) planes[q][pl] = 0u;
        xsum[q] = 0;
        for (int tap = 0; tap < 9; ++tap) {
            const int yy = y + tap / 3 - 1, xx = x + tap % 3 - 1;
            if (yy < 0 || yy >= p.H || xx < 0 || xx >= p.W) continue;
            const uint8_t *px = p.act + ((b * p.H + yy) * p.W + xx) * p.Cin;
            for (int c = 0; c < p.Cin; ++c) {
                const uint32_t v = px[c];
                xsum[q] += (int32_t)v;
                const int bitpos = tap * p.Cin + c;
#pragma unroll
                for (int pl = 0; pl < 8; ++pl) planes[q][pl] |= ((v >> pl) & 1u) << bitpos;
            }
        }
    }
    const int64_t Cw_out = (p.Cout + 31) / 32;
    uint32_t word = 0u;
    for (int64_t n = 0; n < p.Cout; ++n) {
        const uint32_t w = wsm[n];
        int32_t best = 0;
        for (int q = 0; q < npix; ++q) {
            int32_t acc = 0;
#pragma unroll
            for (int pl = 0; pl < 8; ++pl) acc += __popc(planes[q][pl] & w) << pl;
            const int32_t s = 2 * acc - xsum[q];
            best = (q == 0) ? s : max(best, s);
        }
        if (p.out_sums) p.out_sums[o * p.Cout + n] = best;
        if (p.out_bits) {
            const uint32_t f = p.flip ? ((p.flip[n >> 5] >> (n & 31)) & 1u) : 0u;
            word |= (((uint32_t)(best >= p.thr[n]) ^ f) & 1u) << (n & 31);
            if ((n & 31) == 31 || n == p.Cout - 1) {
                p.out_bits[o * Cw_out + (n >> 5)] = word;
                word = 0u;
            }
        }
    }
}

}  // namespace

extern "C" int bnn_binary_conv2d(bnn_ctx *ctx, const uint32_t *act, const uint8_t *act_u8, int64_t B, int64_t H,
                                 int64_t W, int64_t C_in, const uint32_t *Wp, int64_t C_out, int pool,
                                 const int32_t *thr, const uint32_t *flip, uint32_t *out_bits, int32_t *out_sums) {
    if (!ctx || B < 0 || H < 0 || W < 0 || C_in < 0 || C_out < 0) return BNN_ERR_INVALID_ARG;
    if (pool != 0 && pool != 1) return BNN_ERR_INVALID_ARG;
    if (H > 32768 || W > 32768) return BNN_ERR_INVALID_ARG;
    if (pool && ((H & 1) || (W & 1))) return BNN_ERR_INVALID_ARG;
    if (B == 0 || H == 0 || W == 0 || C_out == 0) return BNN_OK;
    if ((act == nullptr) == (act_u8 == nullptr)) return BNN_ERR_INVALID_ARG;
    if (!Wp || (!out_bits && !out_sums)) return BNN_ERR_INVALID_ARG;
    if (out_bits && !thr) return BNN_ERR_INVALID_ARG;
    bnn_device_guard guard(ctx);
    if (!guard.ok) return BNN_ERR_CUDA;

    if (act_u8) {
        if (C_in < 1 || 9 * C_in > 32 || C_out > 8192) return BNN_ERR_INVALID_ARG;
        {
            // tensor-core engine: im2col of the image to 32-byte rows (unsigned bytes) times the filters as +-1 bytes
            int TH, TB;
            const bool tiling = bnn_umma_conv_tiling(H, W, pool, &TH, &TB);
            if (ctx->engine != BNN_ENGINE_POPC && bnn_umma_first_conv_ok(B * H * W, C_out) && (tiling || !pool) &&
                !(pool && out_sums)) {
                const size_t a_bytes = ((size_t)B * H * W * 32 + 255) & ~size_t(255);
                const size_t w_bytes = bnn_umma_operand_bytes(C_out, 9 * C_in);
                // the one-word-per-filter operand must be readable as a packed matrix row: 4-byte stride is not 16-byte
                // aligned, so the filters are expanded with a leading dimension of one word
                if (ctx->ws && ctx->ws_bytes >= a_bytes + w_bytes) {
                    uint8_t *A8 = static_cast<uint8_t *>(ctx->ws);
                    int8_t *W8 = reinterpret_cast<int8_t *>(A8 + a_bytes);
                    if (int st = bnn_umma_im2col_u8(ctx, act_u8, B, H, W, C_in, A8)) return st;
                    if (int st = bnn_umma_expand(ctx, Wp, 1, C_out, 9 * C_in, W8)) return st;
                    return bnn_umma_gemm(ctx, A8, 32, true, W8, bnn_umma_operand_ld(9 * C_in), B * H * W, C_out, 9 * C_in, out_sums,
                                         C_out, thr, flip, out_bits, (C_out + 31) / 32, nullptr, 0, pool, H, W);
                }
                if (ctx->engine == BNN_ENGINE_TENSOR) return BNN_ERR_WORKSPACE;
            }
        }
        ConvU8Args a{act_u8, B, (int)H, (int)W, (int)C_in, Wp, C_out, pool, thr, flip, out_bits, out_sums};
        const int64_t total = B * (pool ? H / 2 : H) * (pool ? W / 2 : W);
        const int64_t blocks = (total + 127) / 128;
        if (blocks > 0x7fffffff) return BNN_ERR_INVALID_ARG;
        k_conv_u8_planes<<<(unsigned)blocks, 128, (size_t)C_out * 4, ctx->stream>>>(a);
        return bnn_check_launch(ctx);
    }

    if (C_in == 0 || (C_in % 32) != 0) return BNN_ERR_INVALID_ARG;
    const int64_t Cw = C_in / 32;
    if (!bnn_aligned16(act) && (Cw % 4) == 0) return BNN_ERR_ALIGNMENT;
    if (!bnn_aligned16(Wp) && (Cw % 4) == 0) return BNN_ERR_ALIGNMENT;
    if (out_bits && !bnn_aligned16(out_bits)) return BNN_ERR_ALIGNMENT;
    if (ctx->filter_repetition)      // Section 3.3: apply only the distinct 2-D filters of every channel (CUDA cores)
        return bnn_fr_conv(ctx, act, B, H, W, C_in, Wp, C_out, pool, thr, flip, out_bits, out_sums);
    {
        // tensor-core engine: activations and weights are expanded to +-1 bytes in the workspace and the convolution
        // runs as 9 * C_in/128 K steps of TMA 4-D loads whose out-of-image halo arrives as zeros
        int TH, TB;
        const bool shape_ok = (C_in % 128) == 0 && bnn_umma_conv_tiling(H, W, pool, &TH, &TB) && !(pool && out_sums) &&
                              bnn_umma_shape_ok(B * H * W, C_out, 9 * C_in);
        if (ctx->engine != BNN_ENGINE_POPC && shape_ok) {
            const size_t a_bytes = bnn_umma_operand_bytes(B * H * W, C_in), w_bytes = bnn_umma_operand_bytes(C_out, 9 * C_in);
            if (ctx->ws && ctx->ws_bytes >= a_bytes + w_bytes) {
                if (ctx->operand_bits != 8 && (C_in % 256) == 0) {
                    // 4-bit operands (one tap and 256 channels per K step): half the bytes, twice the MMA rate
                    uint8_t *act4 = static_cast<uint8_t *>(ctx->ws);
                    uint8_t *W4 = act4 + bnn_umma_operand_bytes_f4(B * H * W, C_in);
                    if (int st = bnn_umma_expand_f4(ctx, act, Cw, B * H * W, C_in, act4)) return st;
                    if (int st = bnn_umma_expand_f4(ctx, Wp, 9 * Cw, C_out, 9 * C_in, W4)) return st;
                    return bnn_umma_conv_f4(ctx, act4, W4, B, H, W, C_in, C_out, pool, thr, flip, out_bits, nullptr, 0, out_sums);
                }
                int8_t *act8 = static_cast<int8_t *>(ctx->ws);
                int8_t *W8 = act8 + a_bytes;
                if (int st = bnn_umma_expand(ctx, act, Cw, B * H * W, C_in, act8)) return st;
                if (int st = bnn_umma_expand(ctx, Wp, 9 * Cw, C_out, 9 * C_in, W8)) return st;
                return bnn_umma_conv(ctx, act8, W8, B, H, W, C_in, C_out, pool, thr, flip, out_bits, out_sums);
            }
            if (ctx->engine == BNN_ENGINE_TENSOR) return BNN_ERR_WORKSPACE;
        }
    }
    Args a{};
    a.A = act; a.lda = 0;
    a.B = Wp; a.ldb = 9 * Cw;
    a.M = B * H * W;          // with pooling the rows are ordered window-major: 4 consecutive rows = one window
    a.N = C_out; a.K = 9 * C_in;
    a.C = out_sums; a.ldc = C_out;
    a.out = out_bits; a.ldo = (C_out + 31) / 32;
    a.thr = thr; a.flip = flip;
    a.H = (int)H; a.W = (int)W; a.Cw = (int)Cw; a.pool = pool;
    return bnn_launch_tile_conv(ctx, a);
}

extern "C" size_t bnn_conv_workspace_bytes(int64_t B, int64_t H, int64_t W, int64_t C_in, int64_t C_out, int pool) {
    int TH, TB;
    if (B <= 0 || H <= 0 || W <= 0 || C_in <= 0 || C_out <= 0) return 0;
    if (9 * C_in <= 32) {   // first layer on 8-bit input: im2col rows + expanded filters
        if (!bnn_umma_first_conv_ok(B * H * W, C_out) || (pool && !bnn_umma_conv_tiling(H, W, pool, &TH, &TB))) return 0;
        return (((size_t)B * H * W * 32 + 255) & ~size_t(255)) + bnn_umma_operand_bytes(C_out, 9 * C_in);
    }
    if ((C_in % 128) != 0) return 0;
    if (!bnn_umma_conv_tiling(H, W, pool, &TH, &TB) || !bnn_umma_shape_ok(B * H * W, C_out, 9 * C_in)) return 0;
    return bnn_umma_operand_bytes(B * H * W, C_in) + bnn_umma_operand_bytes(C_out, 9 * C_in);
}

// ---------------------------------------------------------------------------------------------------------
// bnn_convnet_forward
namespace {

inline size_t r256(size_t b) { return (b + 255) & ~size_t(255); }

struct ConvPlan {
    bool chain;            // every layer runs on the tensor engine and hands +-1 bytes to the next one
    size_t bits_bytes;     // one packed activation buffer (two of them)
    size_t act8_bytes;     // one byte activation buffer (two of them, chain only)
    size_t im2col_bytes;   // first layer's 32-byte rows (chain only)
    size_t w8_bytes;       // scratch for one layer's expanded weights (chain only)
};

int plan_convnet(const bnn_ctx *ctx, const bnn_convnet_desc *net, int64_t B, int64_t H, int64_t W, ConvPlan *plan) {
    if (!net || net->n_layers < 1 || !net->layers || B <= 0 || H <= 0 || W <= 0) return BNN_ERR_INVALID_ARG;
    ConvPlan p{};
    p.chain = !ctx || ctx->engine != BNN_ENGINE_POPC;
    int64_t h = H, w = W;
    for (int k = 0; k < net->n_layers; ++k) {
        const bnn_conv_layer_desc &L = net->layers[k];
        if (L.C_in <= 0 || L.C_out <= 0 || !L.Wp || !L.thr || (L.pool != 0 && L.pool != 1)) return BNN_ERR_INVALID_ARG;
        if (k == 0 ? (9 * L.C_in > 32) : (L.C_in != net->layers[k - 1].C_out || (L.C_in % 32) != 0)) return BNN_ERR_INVALID_ARG;
        if (L.pool && ((h & 1) || (w & 1))) return BNN_ERR_INVALID_ARG;
        int TH, TB;
        const bool tiling = bnn_umma_conv_tiling(h, w, L.pool, &TH, &TB);
        if (k == 0) {
            if (!tiling || !bnn_umma_first_conv_ok(B * h * w, L.C_out)) p.chain = false;
            p.im2col_bytes = r256((size_t)B * h * w * 32);
        } else {
            if (!tiling || (L.C_in % 128) != 0 || !bnn_umma_shape_ok(B * h * w, L.C_out, 9 * L.C_in)) p.chain = false;
        }
        if (k < net->n_layers - 1 && (L.C_out % 128) != 0) p.chain = false;      // the next layer reads these bytes with TMA
        const size_t w8 = bnn_umma_operand_bytes(L.C_out, 9 * L.C_in);
        p.w8_bytes = w8 > p.w8_bytes ? w8 : p.w8_bytes;
        const int64_t ho = L.pool ? h / 2 : h, wo = L.pool ? w / 2 : w;
        const size_t bits = r256((size_t)B * ho * wo * ((L.C_out + 31) / 32) * 4);
        const size_t a8 = r256((size_t)B * ho * wo * L.C_out);
        p.bits_bytes = bits > p.bits_bytes ? bits : p.bits_bytes;
        p.act8_bytes = a8 > p.act8_bytes ? a8 : p.act8_bytes;
        h = ho; w = wo;
    }
    *plan = p;
    return BNN_OK;
}

size_t plan_bytes(const ConvPlan &p) {
    // sized for the tensor engine whenever the shapes allow it, whatever engine is selected later
    return 2 * p.bits_bytes + (p.chain ? 2 * p.act8_bytes + p.im2col_bytes + p.w8_bytes : 0);
}

}  // namespace

extern "C" size_t bnn_convnet_workspace_bytes(const bnn_convnet_desc *net, int64_t B, int64_t H, int64_t W) {
    ConvPlan p;
    if (plan_convnet(nullptr, net, B, H, W, &p) != BNN_OK) return 0;
    return plan_bytes(p);
}

extern "C" int bnn_convnet_forward(bnn_ctx *ctx, const bnn_convnet_desc *net, const uint8_t *X, int64_t B, int64_t H, int64_t W,
                                   uint32_t *out_bits, uint32_t *const *layer_out) {
    if (!ctx || B < 0 || H < 0 || W < 0) return BNN_ERR_INVALID_ARG;
    if (B == 0 || H == 0 || W == 0) return (net && net->n_layers >= 1 && net->layers) ? BNN_OK : BNN_ERR_INVALID_ARG;
    ConvPlan full, plan;
    if (int st = plan_convnet(nullptr, net, B, H, W, &full)) return st;
    if (int st = plan_convnet(ctx, net, B, H, W, &plan)) return st;
    if (!X || !out_bits) return BNN_ERR_INVALID_ARG;
    if (!ctx->ws || ctx->ws_bytes < plan_bytes(full)) return BNN_ERR_WORKSPACE;
    if (ctx->engine == BNN_ENGINE_TENSOR && !plan.chain) return BNN_ERR_INVALID_ARG;   // forced engine, unsuitable shapes
    bnn_device_guard guard(ctx);
    if (!guard.ok) return BNN_ERR_CUDA;

    char *ws = static_cast<char *>(ctx->ws);
    uint32_t *bits[2] = {reinterpret_cast<uint32_t *>(ws), reinterpret_cast<uint32_t *>(ws + full.bits_bytes)};
    int8_t *act8[2] = {reinterpret_cast<int8_t *>(ws + 2 * full.bits_bytes),
                       reinterpret_cast<int8_t *>(ws + 2 * full.bits_bytes + full.act8_bytes)};
    uint8_t *im2col = reinterpret_cast<uint8_t *>(ws + 2 * full.bits_bytes + 2 * full.act8_bytes);
    int8_t *w8_scratch = reinterpret_cast<int8_t *>(ws + 2 * full.bits_bytes + 2 * full.act8_bytes + full.im2col_bytes);
    const int L = net->n_layers;
    int64_t h = H, w = W;

    if (!plan.chain) {
        // one bnn_binary_conv2d per layer on the CUDA-core kernels (they must not expand into the workspace the
        // activations live in, so the engine is pinned for the duration)
        const int saved = ctx->engine;
        ctx->engine = BNN_ENGINE_POPC;
        int st = BNN_OK;
        const uint32_t *cur = nullptr;
        for (int k = 0; k < L && st == BNN_OK; ++k) {
            const bnn_conv_layer_desc &D = net->layers[k];
            uint32_t *dst = (k == L - 1) ? out_bits : bits[k & 1];
            st = bnn_binary_conv2d(ctx, k == 0 ? nullptr : cur, k == 0 ? X : nullptr, B, h, w, D.C_in, D.Wp, D.C_out, D.pool,
                                   D.thr, D.flip, dst, nullptr);
            if (D.pool) { h /= 2; w /= 2; }
            if (st == BNN_OK && layer_out && layer_out[k] && layer_out[k] != dst) {
                cudaError_t e = cudaMemcpyAsync(layer_out[k], dst, (size_t)B * h * w * ((D.C_out + 31) / 32) * 4,
                                                cudaMemcpyDeviceToDevice, ctx->stream);
                if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; st = BNN_ERR_CUDA; }
            }
            cur = dst;
        }
        ctx->engine = saved;
        return st;
    }

    // A layer with a multiple of 256 input channels, or with exactly 128 where the halo-tile kernel takes it, runs on 4-bit
    // operands (e2m1 nibbles, twice the MMA rate and half the operand bytes; a K step is one tap and 256 or 128 channels);
    // the layer before it then writes nibbles instead of bytes.
    auto on_nibbles = [&](int k) {
        if (k <= 0 || k >= L || ctx->operand_bits == 8) return false;
        int64_t hk = H, wk = W;                                      // the layer's input size
        for (int i = 0; i < k; ++i) if (net->layers[i].pool) { hk /= 2; wk /= 2; }
        return bnn_umma_conv_f4_takes(ctx, hk, wk, net->layers[k].pool, net->layers[k].C_in);
    };
    const int8_t *cur8 = nullptr;
    for (int k = 0; k < L; ++k) {
        const bnn_conv_layer_desc &D = net->layers[k];
        uint32_t *dst = (k == L - 1) ? out_bits : bits[k & 1];
        int8_t *dst8 = (k < L - 1) ? act8[k & 1] : nullptr;
        const int next_f4 = on_nibbles(k + 1) ? 1 : 0;
        const int64_t ldo8 = next_f4 ? D.C_out / 2 : D.C_out;
        // an inner layer's packed map is only written when the caller asked for it (the next layer reads the bytes);
        // the pooling epilogue always goes through it
        if (k < L - 1 && !D.pool && !(layer_out && layer_out[k])) dst = nullptr;
        int st;
        if (on_nibbles(k)) {
            const uint8_t *W4 = D.W4;
            if (!W4) {
                uint8_t *w4_scratch = reinterpret_cast<uint8_t *>(w8_scratch);      // half the size of the byte form
                if ((st = bnn_umma_expand_f4(ctx, D.Wp, 9 * (D.C_in / 32), D.C_out, 9 * D.C_in, w4_scratch))) return st;
                W4 = w4_scratch;
            }
            st = bnn_umma_conv_f4(ctx, reinterpret_cast<const uint8_t *>(cur8), W4, B, h, w, D.C_in, D.C_out, D.pool, D.thr, D.flip, dst,
                                  reinterpret_cast<uint8_t *>(dst8), ldo8, nullptr, D.W4 ? 1 : 0);
        } else {
            const int8_t *W8 = D.W8;
            if (!W8) {
                // first layer: one word per filter; others: C_out rows of 9 * C_in bits
                if ((st = bnn_umma_expand(ctx, D.Wp, k == 0 ? 1 : 9 * (D.C_in / 32), D.C_out, 9 * D.C_in, w8_scratch))) return st;
                W8 = w8_scratch;
            }
            if (k == 0) {
                if ((st = bnn_umma_im2col_u8(ctx, X, B, h, w, D.C_in, im2col))) return st;
                st = bnn_umma_gemm(ctx, im2col, 32, true, W8, bnn_umma_operand_ld(9 * D.C_in), B * h * w, D.C_out, 9 * D.C_in, nullptr, 0,
                                   D.thr, D.flip, dst, (D.C_out + 31) / 32, dst8, ldo8, D.pool, h, w, next_f4);
            } else {
                st = bnn_umma_conv(ctx, cur8, W8, B, h, w, D.C_in, D.C_out, D.pool, D.thr, D.flip, dst, nullptr, dst8, ldo8, next_f4, D.W8 ? 1 : 0);
            }
        }
        if (st) return st;
        if (D.pool) { h /= 2; w /= 2; }
        if (dst && layer_out && layer_out[k] && layer_out[k] != dst)
            BNN_CUDA_TRY(ctx, cudaMemcpyAsync(layer_out[k], dst, (size_t)B * h * w * ((D.C_out + 31) / 32) * 4,
                                              cudaMemcpyDeviceToDevice, ctx->stream));
        cur8 = dst8;
    }
    return BNN_OK;
}
