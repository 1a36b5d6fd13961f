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
    {
        // tensor-core engine: activations and weights are expanded to +-1 bytes in the workspace and the convolution
        // runs as 9 * C_in/128 K steps of TMA 4-D loads whose out-of-image halo arrives as zeros
        int TH, TB;
        const bool shape_ok = (C_in % 128) == 0 && bnn_umma_conv_tiling(H, W, pool, &TH, &TB) && !(pool && out_sums) &&
                              bnn_umma_shape_ok(B * H * W, C_out, 9 * C_in);
        if (ctx->engine != BNN_ENGINE_POPC && shape_ok) {
            const size_t a_bytes = bnn_umma_operand_bytes(B * H * W, C_in), w_bytes = bnn_umma_operand_bytes(C_out, 9 * C_in);
            if (ctx->ws && ctx->ws_bytes >= a_bytes + w_bytes) {
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
