// bnn_pack_signs: Sign (Eq. 1) followed by 32-per-word concatenation (Section 4).  Pure streaming.
#include "bnn_common.cuh"
#include <cuda_fp16.h>

namespace {

template <typename T> __device__ __forceinline__ bool is_plus(T v);
template <> __device__ __forceinline__ bool is_plus<float>(float v) { return v >= 0.0f; }
template <> __device__ __forceinline__ bool is_plus<__half>(__half v) { return __half2float(v) >= 0.0f; }
template <> __device__ __forceinline__ bool is_plus<int8_t>(int8_t v) { return v >= 0; }

// Pack along the contiguous axis.  One warp produces WPW consecutive words of one row per step:
// lane l reads element 32*w + l of each word (coalesced), one ballot per word.
template <typename T, int WPW>
__global__ void __launch_bounds__(256) k_pack_cols(const T *__restrict__ src, int64_t rows, int64_t cols,
                                                   int64_t src_ld, uint32_t *__restrict__ dst, int64_t dst_ld) {
    const int lane = threadIdx.x & 31;
    const int64_t warps_per_row = (dst_ld + WPW - 1) / WPW;
    const int64_t total = rows * warps_per_row;
    for (int64_t wi = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); wi < total;
         wi += (int64_t)gridDim.x * (blockDim.x >> 5)) {
        const int64_t r = wi / warps_per_row;
        const int64_t w0 = (wi - r * warps_per_row) * WPW;
        const T *row = src + r * src_ld;
        bool p[WPW];
#pragma unroll
        for (int j = 0; j < WPW; ++j) {
            const int64_t c = (w0 + j) * 32 + lane;
            p[j] = (c < cols) ? is_plus<T>(row[c]) : false;
        }
        uint32_t mine = 0;
#pragma unroll
        for (int j = 0; j < WPW; ++j) {
            const uint32_t word = __ballot_sync(0xffffffffu, p[j]);
            if (lane == j) mine = word;
        }
        if (lane < WPW && w0 + lane < dst_ld) dst[r * dst_ld + w0 + lane] = mine;
    }
}

// int8 source, 4 elements per lane per load (128 contiguous bytes per warp); each lane turns its
// 4 bytes into a nibble and the 8 lanes that share a word OR their nibbles together.
__global__ void __launch_bounds__(256) k_pack_cols_i8x4(const int8_t *__restrict__ src, int64_t rows, int64_t cols,
                                                        int64_t src_ld, uint32_t *__restrict__ dst,
                                                        int64_t dst_ld) {
    const int lane = threadIdx.x & 31;
    const int64_t groups_per_row = (dst_ld + 3) / 4;   // 4 words = 128 elements per warp step
    const int64_t total = rows * groups_per_row;
    for (int64_t wi = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); wi < total;
         wi += (int64_t)gridDim.x * (blockDim.x >> 5)) {
        const int64_t r = wi / groups_per_row;
        const int64_t w0 = (wi - r * groups_per_row) * 4;
        const int64_t c0 = w0 * 32 + lane * 4;
        uint32_t v = 0x80808080u;                      // four negative bytes = four 0 bits
        if (c0 + 3 < cols) {
            v = *reinterpret_cast<const uint32_t *>(src + r * src_ld + c0);
        } else {
#pragma unroll
            for (int b = 0; b < 4; ++b)
                if (c0 + b < cols) {
                    const uint32_t byte = (uint8_t)src[r * src_ld + c0 + b];
                    v = (v & ~(0xffu << (8 * b))) | (byte << (8 * b));
                }
        }
        const uint32_t plus = (~v) & 0x80808080u;      // bit 7 of each byte clear <=> value >= 0
        uint32_t nib = ((plus >> 7) * 0x01020408u) >> 24;   // gather bits 0,8,16,24 into bits 0..3
        nib = (nib & 0xfu) << (4 * (lane & 7));
        nib |= __shfl_xor_sync(0xffffffffu, nib, 1);
        nib |= __shfl_xor_sync(0xffffffffu, nib, 2);
        nib |= __shfl_xor_sync(0xffffffffu, nib, 4);
        if ((lane & 7) == 0 && w0 + (lane >> 3) < dst_ld) dst[r * dst_ld + w0 + (lane >> 3)] = nib;
    }
}

// float32 / float16 source, 16 bytes per lane per load (4 or 8 elements, 512 contiguous bytes per warp, two loads in
// flight): each lane turns its elements into VEC bits, the LPW lanes that share a word OR them together.
template <typename T>
__global__ void __launch_bounds__(256) k_pack_cols_vec(const T *__restrict__ src, int64_t rows, int64_t cols, int64_t src_ld,
                                                       uint32_t *__restrict__ dst, int64_t dst_ld) {
    constexpr int VEC = 16 / (int)sizeof(T), LPW = 32 / VEC, WPS = 32 / LPW;   // elements per lane, lanes per word, words per step
    const int lane = threadIdx.x & 31;
    const int64_t groups_per_row = (dst_ld + WPS - 1) / WPS;
    const int64_t total = rows * groups_per_row;
    const int64_t stride = (int64_t)gridDim.x * (blockDim.x >> 5);
    constexpr int UNR = 4;                  // loads in flight per warp
    for (int64_t wi = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); wi < total; wi += UNR * stride) {
        union { uint4 q; T e[VEC]; } v[UNR];
        int64_t r[UNR], w0[UNR];
        bool live[UNR];
        int nvalid[UNR];
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const int64_t wj = wi + u * stride;
            live[u] = wj < total;
            r[u] = live[u] ? wj / groups_per_row : 0;
            w0[u] = live[u] ? (wj - r[u] * groups_per_row) * WPS : 0;
            const int64_t c0 = w0[u] * 32 + lane * VEC;
            nvalid[u] = 0;
            v[u].q = make_uint4(0u, 0u, 0u, 0u);
            if (live[u] && c0 < cols) {
                const T *ptr = src + r[u] * src_ld + c0;
                if (c0 + VEC <= cols) {
                    v[u].q = *reinterpret_cast<const uint4 *>(ptr);
                    nvalid[u] = VEC;
                } else {
                    nvalid[u] = (int)(cols - c0);
#pragma unroll
                    for (int b = 0; b < VEC; ++b)            // static indices keep the vector in registers
                        if (b < nvalid[u]) v[u].e[b] = ptr[b];
                }
            }
        }
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            uint32_t bits = 0u;
#pragma unroll
            for (int b = 0; b < VEC; ++b) bits |= (uint32_t)(b < nvalid[u] && is_plus<T>(v[u].e[b])) << b;
            bits <<= VEC * (lane % LPW);
#pragma unroll
            for (int d = 1; d < LPW; d <<= 1) bits |= __shfl_xor_sync(0xffffffffu, bits, d);
            if (live[u] && (lane % LPW) == 0 && w0[u] + lane / LPW < dst_ld) dst[r[u] * dst_ld + w0[u] + lane / LPW] = bits;
        }
    }
}

// int8 source, 16 elements per lane per load (512 contiguous bytes per warp, two such loads in flight): each lane turns
// its 16 bytes into 16 bits, lane pairs join them into a word, even lanes store 16 consecutive words.
__device__ __forceinline__ uint32_t plus_bits_of_word(uint32_t v) {
    const uint32_t plus = (~v) & 0x80808080u;              // bit 7 of each byte clear <=> value >= 0
    return (((plus >> 7) * 0x01020408u) >> 24) & 0xfu;      // gather bits 0, 8, 16, 24 into bits 0..3
}
__global__ void __launch_bounds__(256) k_pack_cols_i8x16(const int8_t *__restrict__ src, int64_t rows, int64_t cols,
                                                         int64_t src_ld, uint32_t *__restrict__ dst, int64_t dst_ld) {
    const int lane = threadIdx.x & 31;
    const int64_t groups_per_row = (dst_ld + 15) / 16;   // 16 words = 512 elements per warp step
    const int64_t total = rows * groups_per_row;
    const int64_t stride = (int64_t)gridDim.x * (blockDim.x >> 5);
    constexpr int UNR = 4;                  // loads in flight per warp
    for (int64_t wi = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); wi < total; wi += UNR * stride) {
        uint4 v[UNR];
        int64_t r[UNR], w0[UNR];
        bool live[UNR];
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const int64_t wj = wi + u * stride;
            live[u] = wj < total;
            r[u] = live[u] ? wj / groups_per_row : 0;
            w0[u] = live[u] ? (wj - r[u] * groups_per_row) * 16 : 0;
            const int64_t c0 = w0[u] * 32 + lane * 16;
            v[u] = make_uint4(0x80808080u, 0x80808080u, 0x80808080u, 0x80808080u);    // negative bytes = 0 bits
            if (live[u]) {
                const int8_t *ptr = src + r[u] * src_ld + c0;
                if (c0 + 16 <= cols) {
                    v[u] = *reinterpret_cast<const uint4 *>(ptr);
                } else if (c0 < cols) {
                    uint32_t t[4] = {0x80808080u, 0x80808080u, 0x80808080u, 0x80808080u};
                    for (int b = 0; b < 16 && c0 + b < cols; ++b)
                        t[b >> 2] = (t[b >> 2] & ~(0xffu << (8 * (b & 3)))) | ((uint32_t)(uint8_t)ptr[b] << (8 * (b & 3)));
                    v[u] = make_uint4(t[0], t[1], t[2], t[3]);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            uint32_t h = plus_bits_of_word(v[u].x) | (plus_bits_of_word(v[u].y) << 4) | (plus_bits_of_word(v[u].z) << 8) |
                         (plus_bits_of_word(v[u].w) << 12);
            const uint32_t other = __shfl_down_sync(0xffffffffu, h, 1);
            if (live[u] && (lane & 1) == 0 && w0[u] + (lane >> 1) < dst_ld) dst[r[u] * dst_ld + w0[u] + (lane >> 1)] = h | (other << 16);
        }
    }
}

// Pack along rows: src is K x N (rows = K), dst is N x ceil(K/32).  A 32 x 32 element block is read
// row by row (coalesced along n), every lane builds the word of its own column, and the 32 words
// are written through shared memory so that each output row receives contiguous words.
template <typename T>
__global__ void __launch_bounds__(256) k_pack_rows(const T *__restrict__ src, int64_t K, int64_t N, int64_t src_ld,
                                                   uint32_t *__restrict__ dst, int64_t dst_ld) {
    // block: 8 warps = 8 consecutive k-words for 32 columns
    __shared__ uint32_t tile[32][9];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t n0 = (int64_t)blockIdx.x * 32;
    const int64_t wbase = (int64_t)blockIdx.y * 8;
    const int64_t n = n0 + lane;
    const int64_t kw = wbase + warp;
    uint32_t word = 0;
    if (n < N && kw * 32 < K) {
#pragma unroll 8
        for (int i = 0; i < 32; ++i) {
            const int64_t k = kw * 32 + i;
            if (k < K && is_plus<T>(src[k * src_ld + n])) word |= (1u << i);
        }
    }
    tile[lane][warp] = word;
    __syncthreads();
    // 256 threads write 32 columns x 8 words: thread -> (column = tid / 8, word = tid % 8)
    const int col = threadIdx.x >> 3, wj = threadIdx.x & 7;
    if (n0 + col < N && wbase + wj < dst_ld) dst[(n0 + col) * dst_ld + wbase + wj] = tile[col][wj];
}

template <typename T>
int launch_pack(bnn_ctx *ctx, const T *src, int64_t rows, int64_t cols, int64_t src_ld, int pack_along,
                uint32_t *dst, int64_t dst_ld) {
    if (pack_along == 0 && sizeof(T) == 2 && (reinterpret_cast<uintptr_t>(src) & 15u) == 0 && (src_ld * sizeof(T)) % 16 == 0) {
        constexpr int WPS = 32 / (32 / (16 / (int)sizeof(T)));
        const int64_t warps = rows * ((dst_ld + WPS - 1) / WPS);
        int64_t blocks = (warps + 31) / 32;      // four steps per warp and pass
        const int64_t cap = (int64_t)ctx->sm_count * 16;
        if (blocks > cap) blocks = cap;
        if (blocks < 1) blocks = 1;
        k_pack_cols_vec<T><<<(unsigned)blocks, 256, 0, ctx->stream>>>(src, rows, cols, src_ld, dst, dst_ld);
    } else if (pack_along == 0) {
        constexpr int WPW = 8;               // eight coalesced loads in flight per warp
        const int64_t warps = rows * ((dst_ld + WPW - 1) / WPW);
        int64_t blocks = (warps + 7) / 8;
        const int64_t cap = (int64_t)ctx->sm_count * 64;
        if (blocks > cap) blocks = cap;
        k_pack_cols<T, WPW><<<(unsigned)blocks, 256, 0, ctx->stream>>>(src, rows, cols, src_ld, dst, dst_ld);
    } else {
        const int64_t K = rows, N = cols;
        dim3 grid((unsigned)((N + 31) / 32), (unsigned)((dst_ld + 7) / 8));
        k_pack_rows<T><<<grid, 256, 0, ctx->stream>>>(src, K, N, src_ld, dst, dst_ld);
    }
    return bnn_check_launch(ctx);
}

}  // namespace

extern "C" int bnn_pack_signs(bnn_ctx *ctx, const void *src, int dtype, int64_t rows, int64_t cols,
                              int64_t src_ld, int pack_along, int word_bits, uint32_t *dst, int64_t dst_ld_w) {
    if (!ctx || rows < 0 || cols < 0) return BNN_ERR_INVALID_ARG;
    if (pack_along != 0 && pack_along != 1) return BNN_ERR_INVALID_ARG;
    if (word_bits != 32 && word_bits != 64) return BNN_ERR_INVALID_ARG;
    if (dtype != BNN_F32 && dtype != BNN_F16 && dtype != BNN_I8) return BNN_ERR_INVALID_ARG;
    const int64_t out_rows = pack_along == 0 ? rows : cols;
    const int64_t out_k = pack_along == 0 ? cols : rows;
    if (out_rows == 0) return BNN_OK;
    if (int st = bnn_check_packed(dst, dst_ld_w, out_k, out_rows)) return st;
    if (out_k > 0 && (!src || src_ld < cols)) return BNN_ERR_INVALID_ARG;
    if (pack_along == 1 && (dst_ld_w + 7) / 8 > 65535) return BNN_ERR_INVALID_ARG;
    bnn_device_guard guard(ctx);
    if (!guard.ok) return BNN_ERR_CUDA;
    if (out_k == 0) {   // nothing to read: all padding
        BNN_CUDA_TRY(ctx, cudaMemsetAsync(dst, 0, (size_t)out_rows * dst_ld_w * 4, ctx->stream));
        return BNN_OK;
    }
    switch (dtype) {
        case BNN_F32: return launch_pack(ctx, static_cast<const float *>(src), rows, cols, src_ld, pack_along, dst, dst_ld_w);
        case BNN_F16: return launch_pack(ctx, static_cast<const __half *>(src), rows, cols, src_ld, pack_along, dst, dst_ld_w);
        default: {
            const int8_t *s8 = static_cast<const int8_t *>(src);
            if (pack_along == 0 && (reinterpret_cast<uintptr_t>(s8) & 15u) == 0 && (src_ld % 16) == 0) {
                const int64_t warps = rows * ((dst_ld_w + 15) / 16);
                int64_t blocks = (warps + 31) / 32;          // four steps per warp and pass
                const int64_t cap = (int64_t)ctx->sm_count * 16;
                if (blocks > cap) blocks = cap;
                if (blocks < 1) blocks = 1;
                k_pack_cols_i8x16<<<(unsigned)blocks, 256, 0, ctx->stream>>>(s8, rows, cols, src_ld, dst, dst_ld_w);
                return bnn_check_launch(ctx);
            }
            if (pack_along == 0 && (reinterpret_cast<uintptr_t>(s8) & 3u) == 0 && (src_ld % 4) == 0) {
                const int64_t warps = rows * ((dst_ld_w + 3) / 4);
                int64_t blocks = (warps + 7) / 8;
                const int64_t cap = (int64_t)ctx->sm_count * 16;
                if (blocks > cap) blocks = cap;
                k_pack_cols_i8x4<<<(unsigned)blocks, 256, 0, ctx->stream>>>(s8, rows, cols, src_ld, dst, dst_ld_w);
                return bnn_check_launch(ctx);
            }
            return launch_pack(ctx, s8, rows, cols, src_ld, pack_along, dst, dst_ld_w);
        }
    }
}
