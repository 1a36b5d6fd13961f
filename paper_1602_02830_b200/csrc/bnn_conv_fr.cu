// Exploiting filter repetitions (Section 3.3): a 3x3 binary filter over C_in channels is C_in two-dimensional 3x3
// filters, and there are only 2^9 of those -- 2^8 when a filter and its negation count as one ("merely a multiplication
// of the original filter by -1").  So per input channel only the DISTINCT 2-D filters among the layer's C_out filters
// are applied to the map, and every 3-D filter's result is a signed sum of those response maps:
//
//   classify   every (filter n, channel c): the 9 weight bits, negated if tap 0 is -1, give a class code in 0..255 and
//              a sign;
//   compact    per channel: the classes that occur, numbered 0 .. U_c - 1;
//   convolve   per tile of 32 output rows and 128 filters, channel by channel: the 9-bit neighbourhood of every pixel,
//              the response of each of the channel's U_c distinct filters to it (valid taps minus twice the popcount of
//              the masked XOR: one XNOR-popcount per distinct 2-D filter and pixel instead of one per filter and pixel),
//              then  acc[n] += sign[n][c] * response[class[n][c]].
//
// Taps outside the image contribute 0, pooling / threshold / Sign / packing as in bnn_binary_conv2d.  This is the
// mechanism on CUDA cores, selected by bnn_set_conv_filter_repetition; it is not a fast path on this GPU (the tensor-core
// engine does the full product faster than this does a third of it), see the benchmark's filter_repetition block.
#include "bnn_internal.cuh"
#include <new>

namespace {

// One thread per (filter, channel).
__global__ void __launch_bounds__(256) k_fr_classify(const uint32_t *__restrict__ Wp, int64_t C_out, int64_t C_in,
                                                     uint8_t *__restrict__ code, uint8_t *__restrict__ neg) {
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= C_out * C_in) return;
    const int64_t n = e / C_in, c = e % C_in, Cw = C_in / 32;
    uint32_t f9 = 0u;
    for (int tap = 0; tap < 9; ++tap) f9 |= ((Wp[(n * 9 + tap) * Cw + (c >> 5)] >> (c & 31)) & 1u) << tap;
    uint32_t negated = 0u;
    if ((f9 & 1u) == 0u) { f9 ^= 0x1ffu; negated = 1u; }      // canonical representative: tap 0 is +1
    code[c * C_out + n] = (uint8_t)(f9 >> 1);
    neg[c * C_out + n] = (uint8_t)negated;
}

// One CTA per channel: which of the 256 classes occur, their numbering, and every filter's number.
__global__ void __launch_bounds__(256) k_fr_compact(const uint8_t *__restrict__ code, int64_t C_out, uint8_t *__restrict__ uidx,
                                                    uint8_t *__restrict__ ulist, int32_t *__restrict__ count) {
    __shared__ int present[256];
    __shared__ int rank[256];
    const int64_t c = blockIdx.x;
    present[threadIdx.x] = 0;
    __syncthreads();
    for (int64_t n = threadIdx.x; n < C_out; n += 256) present[code[c * C_out + n]] = 1;
    __syncthreads();
    if (threadIdx.x == 0) {
        int r = 0;
        for (int k = 0; k < 256; ++k) { rank[k] = r; if (present[k]) { ulist[c * 256 + r] = (uint8_t)k; ++r; } }
        count[c] = r;
    }
    __syncthreads();
    for (int64_t n = threadIdx.x; n < C_out; n += 256) uidx[c * C_out + n] = (uint8_t)rank[code[c * C_out + n]];
}

struct FrArgs {
    const uint32_t *act; int64_t B; int H, W; int64_t C_in, C_out;
    const uint8_t *uidx, *neg, *ulist; const int32_t *count;
    int pool;
    const int32_t *thr; const uint32_t *flip;
    uint32_t *out_bits; int32_t *out_sums;
};

// grid.x: tiles of 32 rows (pixels; with pooling 8 windows of 4 pixels each), grid.y: blocks of 128 filters.
__global__ void __launch_bounds__(128) k_fr_conv(const FrArgs p) {
    __shared__ int8_t resp[256][32];
    __shared__ uint32_t nb[32], vmask[32];
    __shared__ int64_t pbase[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t Cw = p.C_in / 32, M = p.B * p.H * p.W;
    const int64_t n = (int64_t)blockIdx.y * 128 + tid;
    if (tid < 32) {
        const int64_t g = (int64_t)blockIdx.x * 32 + tid;
        int64_t b = 0; int y = 0, x = 0; bool valid = g < M;
        if (valid) {
            if (p.pool) {      // rows in window-major order: 4 consecutive rows = one 2x2 window
                const int64_t w = g >> 2; const int j = (int)(g & 3);
                const int Wo = p.W / 2, Ho = p.H / 2;
                b = w / ((int64_t)Wo * Ho);
                const int wy = (int)((w / Wo) % Ho), wx = (int)(w % Wo);
                y = 2 * wy + (j >> 1); x = 2 * wx + (j & 1);
            } else {
                b = g / ((int64_t)p.H * p.W);
                y = (int)((g / p.W) % p.H); x = (int)(g % p.W);
            }
        }
        uint32_t vm = 0u;
        if (valid)
            for (int tap = 0; tap < 9; ++tap) {
                const int yy = y + tap / 3 - 1, xx = x + tap % 3 - 1;
                if (yy >= 0 && yy < p.H && xx >= 0 && xx < p.W) vm |= 1u << tap;
            }
        vmask[tid] = vm;
        pbase[tid] = ((b * p.H + y) * p.W + x) * Cw;
    }
    int32_t acc[32];
#pragma unroll
    for (int r = 0; r < 32; ++r) acc[r] = 0;
    for (int64_t c = 0; c < p.C_in; ++c) {
        __syncthreads();
        if (tid < 32) {      // the pixel's 3x3 neighbourhood in channel c as 9 bits (taps outside the image: 0, masked below)
            uint32_t a9 = 0u;
            const uint32_t vm = vmask[tid];
            for (int tap = 0; tap < 9; ++tap)
                if ((vm >> tap) & 1u) {
                    const int64_t off = ((int64_t)(tap / 3 - 1) * p.W + (tap % 3 - 1)) * Cw;
                    a9 |= ((p.act[pbase[tid] + off + (c >> 5)] >> (c & 31)) & 1u) << tap;
                }
            nb[tid] = a9;
        }
        __syncthreads();
        const int U = p.count[c];
        for (int e = tid; e < U * 32; e += 128) {
            const int k = e >> 5, r = e & 31;
            const uint32_t f9 = ((uint32_t)p.ulist[c * 256 + k] << 1) | 1u;
            const uint32_t vm = vmask[r];
            resp[k][r] = (int8_t)(__popc(vm) - 2 * __popc((nb[r] ^ f9) & vm));      // agreements minus disagreements over valid taps
        }
        __syncthreads();
        if (n < p.C_out) {
            const int k = p.uidx[c * p.C_out + n];
            const int sgn = p.neg[c * p.C_out + n] ? -1 : 1;
#pragma unroll
            for (int r = 0; r < 32; ++r) acc[r] += sgn * (int)resp[k][r];
        }
    }
    const int64_t Cw_out = (p.C_out + 31) / 32;
    const int rows_out = p.pool ? 8 : 32;
    const int32_t thr = (p.thr && n < p.C_out) ? p.thr[n] : 0;
    const uint32_t fl = (p.flip && n < p.C_out) ? ((p.flip[n >> 5] >> (n & 31)) & 1u) : 0u;
    const int64_t rows_total = p.pool ? M / 4 : M;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        if (j >= rows_out) break;                        // (8 pooled rows or 32 plain ones; the accumulators stay in registers)
        const int32_t v = p.pool ? max(max(acc[(4 * j) & 31], acc[(4 * j + 1) & 31]), max(acc[(4 * j + 2) & 31], acc[(4 * j + 3) & 31])) : acc[j];
        const int64_t orow = (int64_t)blockIdx.x * rows_out + j;
        if (orow < rows_total) {                         // uniform over the CTA
            if (p.out_sums && n < p.C_out) p.out_sums[orow * p.C_out + n] = v;
            if (p.out_bits) {
                const bool bit = (n < p.C_out) && (((uint32_t)(v >= thr) ^ fl) & 1u);
                const uint32_t word = __ballot_sync(0xffffffffu, bit);
                const int64_t wi = (int64_t)blockIdx.y * 4 + warp;
                if (lane == 0 && wi < Cw_out) p.out_bits[orow * Cw_out + wi] = word;
            }
        }
    }
}

inline size_t r256(size_t b) { return (b + 255) & ~size_t(255); }

}  // namespace

size_t bnn_fr_workspace_bytes(int64_t C_in, int64_t C_out) {
    return 3 * r256((size_t)C_in * C_out) + r256((size_t)C_in * 256) + r256((size_t)C_in * 4);
}

// Classifies and compacts the filters of one layer into `ws`; the tables stay there for bnn_fr_conv.
static int fr_prepare(bnn_ctx *ctx, const uint32_t *Wp, int64_t C_in, int64_t C_out, char *ws, uint8_t **uidx, uint8_t **neg,
                      uint8_t **ulist, int32_t **count) {
    const size_t t = r256((size_t)C_in * C_out);
    uint8_t *code = reinterpret_cast<uint8_t *>(ws);
    *neg = reinterpret_cast<uint8_t *>(ws + t);
    *uidx = reinterpret_cast<uint8_t *>(ws + 2 * t);
    *ulist = reinterpret_cast<uint8_t *>(ws + 3 * t);
    *count = reinterpret_cast<int32_t *>(ws + 3 * t + r256((size_t)C_in * 256));
    const int64_t blocks = (C_in * C_out + 255) / 256;
    if (blocks > 0x7fffffff || C_in > 0x7fffffff) return BNN_ERR_INVALID_ARG;
    k_fr_classify<<<(unsigned)blocks, 256, 0, ctx->stream>>>(Wp, C_out, C_in, code, *neg);
    if (int st = bnn_check_launch(ctx)) return st;
    k_fr_compact<<<(unsigned)C_in, 256, 0, ctx->stream>>>(code, C_out, *uidx, *ulist, *count);
    return bnn_check_launch(ctx);
}

int bnn_fr_conv(bnn_ctx *ctx, const uint32_t *act, int64_t B, int64_t H, int64_t W, int64_t C_in, const uint32_t *Wp, int64_t C_out,
                int pool, const int32_t *thr, const uint32_t *flip, uint32_t *out_bits, int32_t *out_sums) {
    if (!ctx->ws || ctx->ws_bytes < bnn_fr_workspace_bytes(C_in, C_out)) return BNN_ERR_WORKSPACE;
    uint8_t *uidx, *neg, *ulist;
    int32_t *count;
    if (int st = fr_prepare(ctx, Wp, C_in, C_out, static_cast<char *>(ctx->ws), &uidx, &neg, &ulist, &count)) return st;
    FrArgs a{act, B, (int)H, (int)W, C_in, C_out, uidx, neg, ulist, count, pool, thr, flip, out_bits, out_sums};
    const int64_t M = B * H * W, tiles = (M + 31) / 32, nblocks = (C_out + 127) / 128;
    if (tiles > 0x7fffffff || nblocks > 65535) return BNN_ERR_INVALID_ARG;
    k_fr_conv<<<dim3((unsigned)tiles, (unsigned)nblocks), 128, 0, ctx->stream>>>(a);
    return bnn_check_launch(ctx);
}

extern "C" size_t bnn_filter_repetition_workspace_bytes(int64_t C_in, int64_t C_out) {
    if (C_in <= 0 || C_out <= 0 || (C_in % 32) != 0) return 0;
    return bnn_fr_workspace_bytes(C_in, C_out);
}

extern "C" int bnn_filter_repetition_count(bnn_ctx *ctx, const uint32_t *Wp, int64_t C_in, int64_t C_out, int64_t *distinct) {
    if (!ctx || !Wp || !distinct || C_in <= 0 || C_out <= 0 || (C_in % 32) != 0) return BNN_ERR_INVALID_ARG;
    if (!ctx->ws || ctx->ws_bytes < bnn_fr_workspace_bytes(C_in, C_out)) return BNN_ERR_WORKSPACE;
    bnn_device_guard guard(ctx);
    if (!guard.ok) return BNN_ERR_CUDA;
    uint8_t *uidx, *neg, *ulist;
    int32_t *count;
    if (int st = fr_prepare(ctx, Wp, C_in, C_out, static_cast<char *>(ctx->ws), &uidx, &neg, &ulist, &count)) return st;
    int32_t *host = new (std::nothrow) int32_t[C_in];
    if (!host) return BNN_ERR_INVALID_ARG;
    cudaError_t e = cudaMemcpyAsync(host, count, sizeof(int32_t) * C_in, cudaMemcpyDeviceToHost, ctx->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
    if (e != cudaSuccess) { delete[] host; ctx->last_cuda_error = (int)e; return BNN_ERR_CUDA; }
    int64_t total = 0;
    for (int64_t c = 0; c < C_in; ++c) total += host[c];
    delete[] host;
    *distinct = total;
    return BNN_OK;
}
