// bnn_xnor_gemm, bnn_binary_dense, bnn_first_layer_bitplanes: host-side checks and kernel selection,
// plus the "skinny" kernel used when one operand has at most 32 rows (batch 1..32, or the 10-way output layer).
#include "bnn_common.cuh"
#include "bnn_tile.cuh"
#include "bnn_internal.cuh"

using namespace bnn_tile;

namespace {

// ------------------------------------------------------------------------------------------------
// Skinny product.  S (small operand, RS <= 32 rows) is kept in shared memory; every warp streams rows
// of the large operand L (one 128-bit load per lane per 128 words) and forms the RS dot products of
// that row.  One CTA covers 32 rows of L, so that a packed output word can be assembled.
//   MODE 0: C[s][l] int32 and/or bits out[s][l/32]         (S = activations, L = weights)
//   MODE 1: scores[l][s] = BatchNorm(dot) as float32        (S = output-layer weights, L = activations)
struct SkinnyArgs {
    const uint32_t *S; int64_t lds_w; int64_t RS;
    const uint32_t *L; int64_t ldl_w; int64_t RL;
    int64_t K;
    int32_t *C; int64_t ldc;
    int c_rows_are_large;   // C[l * ldc + s] (the small operand supplies the columns) instead of C[s * ldc + l]
    uint32_t *out; int64_t ldo;
    const int32_t *thr; const uint32_t *flip;
    float *scores; int64_t ld_scores;
    const float *gamma, *beta, *mean, *var; double eps;
};

// Sums V per-lane values over the 32 lanes of a warp with V-1 + (5 - log2 V) shuffles for V < 32 (31 per group of
// 32 values otherwise) instead of 5 per value: at every stage half of the values travel to the partner lane.
// On return, for V >= 32 lane l holds the total of value 32*g + l in v[g]; for V < 32 every lane holds the total
// of value l >> (5 - log2 V) in v[0].
template <int N, int O>
__device__ __forceinline__ void butterfly_stage(int32_t *v, int lane) {
    const bool up = (lane & O) != 0;
#pragma unroll
    for (int i = 0; i < N / 2; ++i) {
        const int32_t send = up ? v[i] : v[i + N / 2];
        const int32_t keep = up ? v[i + N / 2] : v[i];
        v[i] = keep + __shfl_xor_sync(0xffffffffu, send, O);
    }
}
template <int V>
__device__ __forceinline__ void warp_sum_many(int32_t (&v)[V], int lane) {
    if constexpr (V >= 32) {
#pragma unroll
        for (int g = 0; g < V / 32; ++g) {
            int32_t *w = &v[32 * g];
            butterfly_stage<32, 16>(w, lane);
            butterfly_stage<16, 8>(w, lane);
            butterfly_stage<8, 4>(w, lane);
            butterfly_stage<4, 2>(w, lane);
            butterfly_stage<2, 1>(w, lane);
            v[g] = w[0];
        }
    } else if constexpr (V == 16) {
        butterfly_stage<16, 16>(v, lane);
        butterfly_stage<8, 8>(v, lane);
        butterfly_stage<4, 4>(v, lane);
        butterfly_stage<2, 2>(v, lane);
        v[0] += __shfl_xor_sync(0xffffffffu, v[0], 1);
    } else {
        static_assert(V == 4, "4, 16 or a multiple of 32 values");
        butterfly_stage<4, 16>(v, lane);
        butterfly_stage<2, 8>(v, lane);
        v[0] += __shfl_xor_sync(0xffffffffu, v[0], 4);
        v[0] += __shfl_xor_sync(0xffffffffu, v[0], 2);
        v[0] += __shfl_xor_sync(0xffffffffu, v[0], 1);
    }
}

template <int RSMAX, int MODE>
__global__ void __launch_bounds__(256, (RSMAX <= 16) ? 3 : 1) k_skinny(const SkinnyArgs p) {
    extern __shared__ __align__(16) uint32_t smem[];
    const int64_t Kw = (p.K + 31) >> 5;
    const int64_t Kw4 = (Kw + 3) & ~int64_t(3);
    uint32_t *Ss = smem;                                           // [RS][Kw4]
    int32_t *res = reinterpret_cast<int32_t *>(smem + p.RS * Kw4);  // [32][RSMAX]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t tail_mask = (p.K & 31) ? ((1u << (p.K & 31)) - 1u) : 0xffffffffu;
    const int64_t l0 = (int64_t)blockIdx.x * 32;
    // Output-layer mode: the small operand and the BatchNorm parameters are weights, not products of the preceding
    // kernel, so they are staged while that kernel still drains; only the activations wait for it.
    if (MODE != 1) { bnn_pdl_wait(); bnn_pdl_launch_next(); }

    // the warp's four rows of the large operand: their first 128-bit chunks are requested before anything else
    const int64_t lrow0 = l0 + warp * 4;
    uint4 b[4];
    if (MODE != 1) {
#pragma unroll
        for (int cc = 0; cc < 4; ++cc)
            b[cc] = load_row_words(p.L + (lrow0 + cc) * p.ldl_w, lrow0 + cc < p.RL, 4 * lane, Kw, tail_mask, true);
    }

    {   // 32-bit index arithmetic: RS <= 32 rows of at most 2^24 128-bit groups
        const uint32_t gpr = (uint32_t)(Kw4 >> 2), total = (uint32_t)p.RS * gpr;
        for (uint32_t e = tid; e < total; e += 256) {
            const uint32_t r = e / gpr, q = e - r * gpr;
            const uint4 v = load_row_words(p.S + (int64_t)r * p.lds_w, true, 4 * (int64_t)q, Kw, tail_mask, true);
            *reinterpret_cast<uint4 *>(Ss + (int64_t)r * Kw4 + 4 * q) = v;
        }
    }
    // thresholds and flip word of the CTA's 32 outputs: requested now, in parallel, so that the packing loop at the end
    // reads shared memory (as 32 dependent global loads of one thread they were half of a batch-1 call's time)
    __shared__ int32_t thr_s[32];
    __shared__ uint32_t flip_s;
    if (MODE == 0 && p.out) {
        if (tid < 32) thr_s[tid] = (l0 + tid < p.RL) ? p.thr[l0 + tid] : 0;
        if (tid == 32) flip_s = p.flip ? p.flip[blockIdx.x] : 0u;
    }
    // output scores: per output s the affine form of BatchNorm, a = gamma / sqrt(var + eps), b = beta - mean * a, once
    // per CTA in double (the square root and the division are the expensive part)
    __shared__ double bn_a[32], bn_b[32];
    if (MODE == 1 && tid < p.RS) {
        const double a = (double)p.gamma[tid] / sqrt((double)p.var[tid] + p.eps);
        bn_a[tid] = a;
        bn_b[tid] = (double)p.beta[tid] - (double)p.mean[tid] * a;
    }
    if (MODE == 1) {
        bnn_pdl_wait();
        bnn_pdl_launch_next();
#pragma unroll
        for (int cc = 0; cc < 4; ++cc)
            b[cc] = load_row_words(p.L + (lrow0 + cc) * p.ldl_w, lrow0 + cc < p.RL, 4 * lane, Kw, tail_mask, true);
    }
    __syncthreads();

    int32_t acc[4 * RSMAX];                                        // value cc * RSMAX + s
#pragma unroll
    for (int e = 0; e < 4 * RSMAX; ++e) acc[e] = 0;
    for (int64_t w4 = 4 * lane; w4 < Kw4; w4 += 128) {
        if (w4 != 4 * lane) {
#pragma unroll
            for (int cc = 0; cc < 4; ++cc)
                b[cc] = load_row_words(p.L + (lrow0 + cc) * p.ldl_w, lrow0 + cc < p.RL, w4, Kw, tail_mask, true);
        }
#pragma unroll
        for (int s = 0; s < RSMAX; ++s) {
            if (s < p.RS) {
                const uint4 a = *reinterpret_cast<const uint4 *>(Ss + s * Kw4 + w4);
#pragma unroll
                for (int cc = 0; cc < 4; ++cc)
                    acc[cc * RSMAX + s] += __popc(a.x ^ b[cc].x) + __popc(a.y ^ b[cc].y) + __popc(a.z ^ b[cc].z) + __popc(a.w ^ b[cc].w);
            }
        }
    }
    warp_sum_many<4 * RSMAX>(acc, lane);
    constexpr int V = 4 * RSMAX;
    if constexpr (V >= 32) {
#pragma unroll
        for (int g = 0; g < V / 32; ++g) {
            const int e = 32 * g + lane, cc = e / RSMAX, sidx = e % RSMAX;
            res[(warp * 4 + cc) * RSMAX + sidx] = (int32_t)p.K - 2 * acc[g];
        }
    } else {
        constexpr int SH = (V == 16) ? 1 : 3;                      // lanes per value
        if ((lane & ((1 << SH) - 1)) == 0) {
            const int e = lane >> SH, cc = e / RSMAX, sidx = e % RSMAX;
            res[(warp * 4 + cc) * RSMAX + sidx] = (int32_t)p.K - 2 * acc[0];
        }
    }
    __syncthreads();

    if (MODE == 0) {
        if (p.C && p.c_rows_are_large) {
            for (int e = tid; e < 32 * (int)p.RS; e += 256) {
                const int lc = e / (int)p.RS, s = e - lc * (int)p.RS;
                if (l0 + lc < p.RL) p.C[(l0 + lc) * p.ldc + s] = res[lc * RSMAX + s];
            }
        } else if (p.C) {
            for (int e = tid; e < 32 * (int)p.RS; e += 256) {
                const int s = e >> 5, lc = e & 31;
                if (l0 + lc < p.RL) p.C[(int64_t)s * p.ldc + l0 + lc] = res[lc * RSMAX + s];
            }
        }
        if (p.out) {
            if (tid < p.RS) {
                uint32_t word = 0u;
                const uint32_t fw = flip_s;
#pragma unroll
                for (int lc = 0; lc < 32; ++lc) {
                    if (l0 + lc < p.RL) {
                        const uint32_t q = res[lc * RSMAX + tid] >= thr_s[lc];
                        word |= ((q ^ (fw >> lc)) & 1u) << lc;
                    }
                }
                p.out[(int64_t)tid * p.ldo + blockIdx.x] = word;
            }
            if (blockIdx.x == gridDim.x - 1) {   // padding words
                const int64_t first_pad = (p.RL + 31) >> 5, npad = p.ldo - first_pad;
                for (int64_t e = tid; e < p.RS * npad; e += 256) p.out[(e / npad) * p.ldo + first_pad + e % npad] = 0u;
            }
        }
    } else {
        for (int e = tid; e < 32 * (int)p.RS; e += 256) {
            const int lc = e / (int)p.RS, s = e % (int)p.RS;
            if (l0 + lc < p.RL) {
                p.scores[(l0 + lc) * p.ld_scores + s] = (float)fma((double)res[lc * RSMAX + s], bn_a[s], bn_b[s]);
            }
        }
    }
}

template <int MODE>
int launch_skinny(bnn_ctx *ctx, const SkinnyArgs &a) {
    const int64_t Kw4 = (bnn_words(a.K) + 3) & ~int64_t(3);
    const int rsmax = a.RS <= 1 ? 1 : (a.RS <= 4 ? 4 : (a.RS <= 16 ? 16 : 32));
    const size_t smem = (size_t)a.RS * Kw4 * 4 + (size_t)32 * rsmax * 4;
    const unsigned grid = (unsigned)((a.RL + 31) / 32);
#define BNN_SK(R)                                                                                              \
    do {                                                                                                       \
        if (smem > 48 * 1024)                                                                                  \
            BNN_CUDA_TRY(ctx, cudaFuncSetAttribute(k_skinny<R, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                                   (int)smem));                                                \
        BNN_CUDA_TRY(ctx, bnn_launch_dependent(k_skinny<R, MODE>, dim3(grid), dim3(256), smem, ctx->stream, a)); \
    } while (0)
    switch (rsmax) {
        case 1: BNN_SK(1); break;
        case 4: BNN_SK(4); break;
        case 16: BNN_SK(16); break;
        default: BNN_SK(32); break;
    }
#undef BNN_SK
    return bnn_check_launch(ctx);
}

bool skinny_fits(int64_t RS, int64_t K) {
    const int64_t Kw4 = (bnn_words(K) + 3) & ~int64_t(3);
    return RS >= 1 && RS <= 32 && (RS * Kw4 * 4 + 32 * 32 * 4) <= 200 * 1024;
}

template <int AKIND>
int launch_tile(bnn_ctx *ctx, const Args &a_in, int variant) {
    Args a = a_in;
    a.one = 1u;
    const int64_t rows = (AKIND == A_PLANES || AKIND == A_PLANES_PRE) ? 8 * a.M : a.M;   // 8 bit-plane rows per image
    const int64_t tn = (a.N + BN - 1) / BN;
    const int64_t t128 = ((rows + 127) / 128) * tn, t64 = ((rows + 63) / 64) * tn;
    const bool csa = (variant != BNN_VARIANT_PLAIN);
    if (t64 > 0x7fffffff) return BNN_ERR_INVALID_ARG;
    if (ctx->tile_rows == 8) {
        // 8 accumulator rows per thread: 64 x 128 tiles, 8 warps, two CTAs per SM
        if (csa) k_bit_tile<8, AKIND, true, 8><<<(unsigned)t64, 256, 0, ctx->stream>>>(a);
        else k_bit_tile<8, AKIND, false, 8><<<(unsigned)t64, 256, 0, ctx->stream>>>(a);
        return bnn_check_launch(ctx);
    }
    const bool big = t128 >= 2 * (int64_t)ctx->sm_count;
    const int64_t tiles = big ? t128 : t64;
    if (big && csa) k_bit_tile<8, AKIND, true, 16><<<(unsigned)tiles, 256, 0, ctx->stream>>>(a);
    else if (big) k_bit_tile<8, AKIND, false, 16><<<(unsigned)tiles, 256, 0, ctx->stream>>>(a);
    else if (csa) k_bit_tile<4, AKIND, true, 16><<<(unsigned)tiles, 128, 0, ctx->stream>>>(a);
    else k_bit_tile<4, AKIND, false, 16><<<(unsigned)tiles, 128, 0, ctx->stream>>>(a);
    return bnn_check_launch(ctx);
}

}  // namespace

// Used by bnn_conv.cu and bnn_mlp.cu.
int bnn_launch_tile_packed(bnn_ctx *ctx, const Args &a) { return launch_tile<A_PACKED>(ctx, a, ctx_variant(ctx)); }
int bnn_launch_tile_conv(bnn_ctx *ctx, const Args &a) { return launch_tile<A_CONV>(ctx, a, ctx_variant(ctx)); }
int bnn_launch_tile_planes(bnn_ctx *ctx, const Args &a) { return launch_tile<A_PLANES>(ctx, a, ctx_variant(ctx)); }

// ------------------------------------------------------------------------------------------------
// Bit-plane split as a pre-pass (Eq. 7): plane p of image m becomes packed row 8*m + p of `planes`, and the sum of
// the image's bytes goes to xsum[m].  One warp per image; lane l handles 32-byte groups l, l+32, ...
namespace {
__global__ void __launch_bounds__(256) k_split_planes(const uint8_t *__restrict__ X, int64_t ldx, int64_t M, int64_t K,
                                                      uint32_t *__restrict__ planes, int64_t ld_w, int32_t *__restrict__ xsum) {
    const int lane = threadIdx.x & 31;
    const int64_t m = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (m >= M) return;
    const uint8_t *row = X + m * ldx;
    int32_t sum = 0;
    for (int64_t w = lane; w < ld_w; w += 32) {
        uint32_t q[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
        const int64_t k0 = 32 * w;
        if (k0 < K) {
            if (k0 + 32 <= K && ((reinterpret_cast<uintptr_t>(row + k0) & 15u) == 0)) {
                const uint4 a = *reinterpret_cast<const uint4 *>(row + k0), b = *reinterpret_cast<const uint4 *>(row + k0 + 16);
                q[0] = a.x; q[1] = a.y; q[2] = a.z; q[3] = a.w; q[4] = b.x; q[5] = b.y; q[6] = b.z; q[7] = b.w;
            } else {
                for (int i = 0; i < 32; ++i)
                    if (k0 + i < K) q[i >> 2] |= (uint32_t)row[k0 + i] << (8 * (i & 3));
            }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) sum += (int32_t)__vsadu4(q[i], 0u);
#pragma unroll
        for (int pl = 0; pl < 8; ++pl) {
            uint32_t word = 0u;
#pragma unroll
            for (int i = 0; i < 8; ++i) word |= plane_nibble(q[i], pl) << (4 * i);
            planes[(8 * m + pl) * ld_w + w] = word;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) xsum[m] = sum;
}
}  // namespace

size_t bnn_planes_scratch_bytes(int64_t M, int64_t K) {
    const int64_t ld_w = ((K + 127) / 128) * 4;
    return (((size_t)8 * M * ld_w * 4 + 255) & ~size_t(255)) + (((size_t)M * 4 + 255) & ~size_t(255));
}

// First layer on the CUDA-core kernels with the split done once into `scratch` (bnn_planes_scratch_bytes).
int bnn_first_layer_planes_pre(bnn_ctx *ctx, const uint8_t *X, int64_t ldx, const uint32_t *Wp, int64_t ldw_w, const int32_t *thr,
                               const uint32_t *flip, uint32_t *out_bits, int64_t ldo_w, int32_t *out_sums, int64_t lds, int64_t M,
                               int64_t N, int64_t K, void *scratch) {
    const int64_t ld_w = ((K + 127) / 128) * 4;
    uint32_t *planes = static_cast<uint32_t *>(scratch);
    int32_t *xsum = reinterpret_cast<int32_t *>(static_cast<char *>(scratch) + (((size_t)8 * M * ld_w * 4 + 255) & ~size_t(255)));
    const int64_t blocks = (M + 7) / 8;
    if (blocks > 0x7fffffff) return BNN_ERR_INVALID_ARG;
    k_split_planes<<<(unsigned)blocks, 256, 0, ctx->stream>>>(X, ldx, M, K, planes, ld_w, xsum);
    if (int st = bnn_check_launch(ctx)) return st;
    Args a{};
    a.A = planes; a.lda = ld_w; a.xsum = xsum; a.B = Wp; a.ldb = ldw_w;
    a.M = M; a.N = N; a.K = K;
    a.C = out_sums; a.ldc = lds; a.out = out_bits; a.ldo = ldo_w; a.thr = thr; a.flip = flip;
    return launch_tile<A_PLANES_PRE>(ctx, a, ctx_variant(ctx));
}

int bnn_output_scores(bnn_ctx *ctx, const uint32_t *Ap, int64_t lda_w, const uint32_t *Wp, int64_t ldw_w,
                      const float *gamma, const float *beta, const float *mean, const float *var, double eps,
                      float *scores, int64_t lds, int64_t M, int64_t N, int64_t K) {
    if (M == 0 || N == 0) return BNN_OK;
    if (!skinny_fits(N, K)) return BNN_ERR_INVALID_ARG;
    SkinnyArgs s{};
    s.S = Wp; s.lds_w = ldw_w; s.RS = N;
    s.L = Ap; s.ldl_w = lda_w; s.RL = M;
    s.K = K;
    s.scores = scores; s.ld_scores = lds;
    s.gamma = gamma; s.beta = beta; s.mean = mean; s.var = var; s.eps = eps;
    return launch_skinny<1>(ctx, s);
}

static int gemm_like(bnn_ctx *ctx, const uint32_t *Ap, int64_t lda_w, const uint32_t *Bp, int64_t ldb_w, int32_t *C,
                     int64_t ldc, const int32_t *thr, const uint32_t *flip, uint32_t *out, int64_t ldo_w, int64_t M,
                     int64_t N, int64_t K) {
    if (!ctx || M < 0 || N < 0 || K < 0 || K > 0x3fffffff) return BNN_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return BNN_OK;
    if (int st = bnn_check_packed(Ap, lda_w, K, K ? M : 0)) return st;
    if (int st = bnn_check_packed(Bp, ldb_w, K, K ? N : 0)) return st;
    if (C) {
        if (ldc < N) return BNN_ERR_INVALID_ARG;
    }
    if (out) {
        if (!thr) return BNN_ERR_INVALID_ARG;
        if (int st = bnn_check_packed(out, ldo_w, N, M)) return st;
    }
    if (!C && !out) return BNN_ERR_INVALID_ARG;
    bnn_device_guard guard(ctx);
    if (!guard.ok) return BNN_ERR_CUDA;
    if (ctx->engine != BNN_ENGINE_POPC && bnn_umma_shape_ok(M, N, K)) {
        // tensor-core engine: both packed operands are expanded to signed bytes in the workspace first
        const size_t need = bnn_umma_operand_bytes(M, K) + bnn_umma_operand_bytes(N, K);
        if (ctx->ws && ctx->ws_bytes >= need) {
            if (ctx->operand_bits == 4 && K <= (1 << 24)) {
                // both operands are +-1: 4-bit (e2m1) operands, exact in the float32 accumulators
                uint8_t *A4 = static_cast<uint8_t *>(ctx->ws);
                uint8_t *B4 = A4 + bnn_umma_operand_bytes_f4(M, K);
                const int64_t ld4 = bnn_umma_operand_ld_f4(K);
                if (int st = bnn_umma_expand_f4(ctx, Ap, lda_w, M, K, A4)) return st;
                if (int st = bnn_umma_expand_f4(ctx, Bp, ldb_w, N, K, B4)) return st;
                return bnn_umma_gemm_f4(ctx, A4, ld4, B4, ld4, M, N, K, C, ldc, thr, flip, out, ldo_w, nullptr, 0);
            }
            int8_t *A8 = static_cast<int8_t *>(ctx->ws);
            int8_t *B8 = A8 + bnn_umma_operand_bytes(M, K);
            const int64_t ld8 = bnn_umma_operand_ld(K);
            if (int st = bnn_umma_expand(ctx, Ap, lda_w, M, K, A8)) return st;
            if (int st = bnn_umma_expand(ctx, Bp, ldb_w, N, K, B8)) return st;
            return bnn_umma_gemm(ctx, A8, ld8, false, B8, ld8, M, N, K, C, ldc, thr, flip, out, ldo_w, nullptr, 0);
        }
        if (ctx->engine == BNN_ENGINE_TENSOR) return BNN_ERR_WORKSPACE;
    }
    if (M <= 32 && skinny_fits(M, K)) {
        SkinnyArgs s{};
        s.S = Ap; s.lds_w = lda_w; s.RS = M;
        s.L = Bp; s.ldl_w = ldb_w; s.RL = N;
        s.K = K;
        s.C = C; s.ldc = ldc; s.out = out; s.ldo = ldo_w; s.thr = thr; s.flip = flip;
        return launch_skinny<0>(ctx, s);
    }
    if (N <= 32 && C && !out && skinny_fits(N, K)) {   // few columns (e.g. a 10-way output layer as a plain product): roles swapped
        SkinnyArgs s{};
        s.S = Bp; s.lds_w = ldb_w; s.RS = N;
        s.L = Ap; s.ldl_w = lda_w; s.RL = M;
        s.K = K;
        s.C = C; s.ldc = ldc; s.c_rows_are_large = 1;
        return launch_skinny<0>(ctx, s);
    }
    Args a{};
    a.A = Ap; a.lda = lda_w; a.B = Bp; a.ldb = ldb_w;
    a.M = M; a.N = N; a.K = K;
    a.C = C; a.ldc = ldc; a.out = out; a.ldo = ldo_w; a.thr = thr; a.flip = flip;
    return bnn_launch_tile_packed(ctx, a);
}

extern "C" int bnn_xnor_gemm(bnn_ctx *ctx, const uint32_t *Ap, int64_t lda_w, const uint32_t *Bp, int64_t ldb_w,
                             int32_t *C, int64_t ldc, int64_t M, int64_t N, int64_t K) {
    if (!C && M > 0 && N > 0) return BNN_ERR_INVALID_ARG;
    return gemm_like(ctx, Ap, lda_w, Bp, ldb_w, C, ldc, nullptr, nullptr, nullptr, 0, M, N, K);
}

extern "C" int bnn_binary_dense(bnn_ctx *ctx, const uint32_t *Ap, int64_t lda_w, const uint32_t *Wp, int64_t ldw_w,
                                const int32_t *thr, const uint32_t *flip, uint32_t *out, int64_t ldo_w, int64_t M,
                                int64_t N, int64_t K) {
    if (!out && M > 0 && N > 0) return BNN_ERR_INVALID_ARG;
    return gemm_like(ctx, Ap, lda_w, Wp, ldw_w, nullptr, 0, thr, flip, out, ldo_w, M, N, K);
}

extern "C" int bnn_binary_dense_expanded(bnn_ctx *ctx, const void *A_exp, int64_t lda_bytes, const void *W_exp, int64_t ldw_bytes,
                                         int operand_bits, const int32_t *thr, const uint32_t *flip, uint32_t *out_bits,
                                         int64_t ldo_w, void *out_exp, int64_t ldo_exp, int64_t M, int64_t N, int64_t K) {
    if (!ctx || M < 0 || N < 0 || K <= 0 || (operand_bits != 4 && operand_bits != 8)) return BNN_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return BNN_OK;
    if (!A_exp || !W_exp || !thr || (!out_bits && !out_exp)) return BNN_ERR_INVALID_ARG;
    const int64_t ld_min = operand_bits == 4 ? bnn_umma_operand_ld_f4(K) : bnn_umma_operand_ld(K);
    if (lda_bytes < ld_min || ldw_bytes < ld_min) return BNN_ERR_INVALID_ARG;
    if (out_bits)
        if (int st = bnn_check_packed(out_bits, ldo_w, N, M)) return st;
    if (out_exp) {
        const int64_t lo_min = operand_bits == 4 ? bnn_umma_operand_ld_f4(N) : bnn_umma_operand_ld(N);
        if (ldo_exp < lo_min) return BNN_ERR_INVALID_ARG;
        if ((ldo_exp & 15) || !bnn_aligned16(out_exp)) return BNN_ERR_ALIGNMENT;
    }
    bnn_device_guard guard(ctx);
    if (!guard.ok) return BNN_ERR_CUDA;
    if (operand_bits == 4)
        return bnn_umma_gemm_f4(ctx, static_cast<const uint8_t *>(A_exp), lda_bytes, static_cast<const uint8_t *>(W_exp), ldw_bytes,
                                M, N, K, nullptr, 0, thr, flip, out_bits, ldo_w, static_cast<uint8_t *>(out_exp), ldo_exp);
    return bnn_umma_gemm(ctx, A_exp, lda_bytes, false, static_cast<const int8_t *>(W_exp), ldw_bytes, M, N, K, nullptr, 0, thr,
                         flip, out_bits, ldo_w, static_cast<int8_t *>(out_exp), ldo_exp);
}

extern "C" int bnn_first_layer_bitplanes(bnn_ctx *ctx, const uint8_t *X, int64_t ldx, const uint32_t *Wp,
                                         int64_t ldw_w, const int32_t *thr, const uint32_t *flip, uint32_t *out_bits,
                                         int64_t ldo_w, int32_t *out_sums, int64_t lds, int64_t M, int64_t N,
                                         int64_t K) {
    if (!ctx || M < 0 || N < 0 || K < 0 || K > (0x7fffffff / 255)) return BNN_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return BNN_OK;
    if (!out_bits && !out_sums) return BNN_ERR_INVALID_ARG;
    if (K > 0 && (!X || ldx < K)) return BNN_ERR_INVALID_ARG;
    if (int st = bnn_check_packed(Wp, ldw_w, K, K ? N : 0)) return st;
    if (out_sums && lds < N) return BNN_ERR_INVALID_ARG;
    if (out_bits) {
        if (!thr) return BNN_ERR_INVALID_ARG;
        if (int st = bnn_check_packed(out_bits, ldo_w, N, M)) return st;
    }
    bnn_device_guard guard(ctx);
    if (!guard.ok) return BNN_ERR_CUDA;
    if (ctx->engine != BNN_ENGINE_POPC && bnn_umma_shape_ok(M, N, K) && (ldx % 16) == 0 && bnn_aligned16(X)) {
        // tensor-core engine: the 8-bit inputs are used as they are (unsigned bytes), only the weights are expanded;
        // the 8 bit-plane products of Eq. 7 collapse into the byte product the tensor core forms in one step
        const size_t need = bnn_umma_operand_bytes(N, K);
        if (ctx->ws && ctx->ws_bytes >= need) {
            int8_t *W8 = static_cast<int8_t *>(ctx->ws);
            if (int st = bnn_umma_expand(ctx, Wp, ldw_w, N, K, W8)) return st;
            return bnn_umma_gemm(ctx, X, ldx, true, W8, bnn_umma_operand_ld(K), M, N, K, out_sums, lds, thr, flip, out_bits,
                                 ldo_w, nullptr, 0);
        }
        if (ctx->engine == BNN_ENGINE_TENSOR) return BNN_ERR_WORKSPACE;
    }
    // CUDA-core path.  With scratch available the bytes are split into bit-planes once (otherwise every column tile
    // of the fused kernel splits its rows again); worth it from a few column tiles on.
    if (N >= 512 && ctx->ws && ctx->ws_bytes >= bnn_planes_scratch_bytes(M, K))
        return bnn_first_layer_planes_pre(ctx, X, ldx, Wp, ldw_w, thr, flip, out_bits, ldo_w, out_sums, lds, M, N, K, ctx->ws);
    Args a{};
    a.X = X; a.ldx = ldx; a.B = Wp; a.ldb = ldw_w;
    a.M = M; a.N = N; a.K = K;
    a.C = out_sums; a.ldc = lds; a.out = out_bits; a.ldo = ldo_w; a.thr = thr; a.flip = flip;
    return bnn_launch_tile_planes(ctx, a);
}

extern "C" size_t bnn_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K) {
    if (M <= 0 || N <= 0 || K <= 0 || !bnn_umma_shape_ok(M, N, K)) return 0;
    return bnn_umma_operand_bytes(M, K) + bnn_umma_operand_bytes(N, K);
}
