// The tiled bit-GEMM kernel every large call of the library runs on (Section 4, Eq. 8).
//
// One CTA computes a BM x 128 tile of outputs.  K is walked in chunks of 8 words (256 bits); a chunk of
// both operands is staged in shared memory transposed to [word][row], so that in the inner loop
//   - the 16 rows a warp owns are fetched as four 128-bit broadcast loads (every lane the same address),
//   - the 4 columns a lane owns (lane, lane+32, lane+64, lane+96) are fetched as conflict-free 32-bit loads,
//   - lane <-> column, so the Sign/repack epilogue is one __ballot_sync per output word.
// Each thread keeps a 16 x 4 block of accumulators in registers.  Global loads of the next chunk are issued
// before the arithmetic of the current one and written to the other shared-memory buffer afterwards.
//
// Inner loops (selected at compile time):
//   PLAIN   acc += popc(a ^ b)                                  1 POPC per word
//   CSA     (ones, carry) = full_add(ones, a0 ^ b0, a1 ^ b1); acc2 += popc(carry)
//           1 POPC per TWO words; the POPC pipe (16 lanes/clk/SM on sm_100) is the bottleneck and
//           the two extra LOP3 go to the 64-lane integer pipe.  Total = 2 * acc2 + popc(ones).
// The accumulate is written as popc * one + acc with `one` a run-time 1, so that it is issued as an integer
// multiply-add on the FMA pipe instead of competing with the LOP3s for the integer pipe.
//
// A-operand sources: a packed matrix; an implicit im2col view of a packed NHWC activation map (3x3, pad 1);
// or an 8-bit matrix split into bit-planes on the fly (Eq. 6-7): each image contributes 8 operand rows, one
// per bit-plane x^p in {0,1}, combined with AND instead of XOR, and the epilogue forms
// s = 2 * sum_p 2^p popc(x^p & w_plus) - sum(x)  (w_plus = the +1 mask of the weights).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace bnn_tile {

constexpr int BN = 128;   // tile columns
constexpr int BKW = 8;    // words of K per chunk
constexpr int TN = 4;     // columns per lane

enum { A_PACKED = 0, A_CONV = 1, A_PLANES = 2, A_PLANES_PRE = 3 };   // PRE: bit-plane rows already split into `A`

struct Args {
    const uint32_t *A;   // A_PACKED: packed M x K; A_CONV: packed NHWC activations
    int64_t lda;
    const uint8_t *X;    // A_PLANES: M x K bytes
    int64_t ldx;
    const uint32_t *B;   // packed N x K
    int64_t ldb;
    int64_t M, N, K;     // K in bits (A_CONV: 9 * C_in; A_PLANES: number of 8-bit inputs)
    int32_t *C;          // optional int32 output
    int64_t ldc;
    uint32_t *out;       // optional packed-bit output
    int64_t ldo;
    const int32_t *thr;
    const uint32_t *flip;
    const int32_t *xsum; // A_PLANES_PRE: sum of the 8-bit inputs of every image
    int H, W, Cw, pool;  // A_CONV geometry: image height/width, C_in/32, 2x2 pooling flag
    uint32_t one;        // always 1; a run-time value so that "popc * one + acc" stays an IMAD
};

__device__ __forceinline__ uint32_t lop3_xor3(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}
__device__ __forceinline__ uint32_t lop3_maj(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, 0xe8;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}

// Four consecutive words of one operand row, with everything at or beyond bit K forced to 0.
__device__ __forceinline__ uint4 load_row_words(const uint32_t *__restrict__ base, bool row_ok, int64_t kw,
                                                int64_t Kw, uint32_t tail_mask, bool vec_ok) {
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row_ok && kw < Kw) {
        if (vec_ok) {
            v = *reinterpret_cast<const uint4 *>(base + kw);
        } else {
            v.x = base[kw];
            if (kw + 1 < Kw) v.y = base[kw + 1];
            if (kw + 2 < Kw) v.z = base[kw + 2];
            if (kw + 3 < Kw) v.w = base[kw + 3];
        }
        const int64_t last = Kw - 1 - kw;   // position of the row's last word inside this quad
        if (last < 4) {
            if (last == 0) { v.x &= tail_mask; v.y = 0u; v.z = 0u; v.w = 0u; }
            else if (last == 1) { v.y &= tail_mask; v.z = 0u; v.w = 0u; }
            else if (last == 2) { v.z &= tail_mask; v.w = 0u; }
            else { v.w &= tail_mask; }
        }
    }
    return v;
}

// Bit p of each of the four bytes of w, gathered into bits 0..3.
__device__ __forceinline__ uint32_t plane_nibble(uint32_t w, int p) {
    return ((((w >> p) & 0x01010101u) * 0x01020408u) >> 24) & 0xfu;
}

// TM = rows per warp (= accumulator rows per thread): 16 (243 registers, one 8-warp CTA per SM) or
// 8 (two CTAs per SM, twice the warps per scheduler to hide the POPC / LOP3 pipe latencies).
template <int NWARPS, int AKIND, bool CSA, int TM>
__global__ void __launch_bounds__(NWARPS * 32, (TM == 8) ? (512 / (NWARPS * 32)) : ((NWARPS == 8) ? 1 : 2)) k_bit_tile(const Args p) {
    constexpr int BM = NWARPS * TM;        // operand rows per tile (A_PLANES: 8 rows per image)
    constexpr int NT = NWARPS * 32;
    static_assert(2 * BM <= NT && (TM == 8 || TM == 16), "at most one A load item per thread");
    constexpr int A_THREADS = 2 * BM;      // threads that load A
    constexpr bool PLANES = (AKIND == A_PLANES) || (AKIND == A_PLANES_PRE);   // 8 AND-popcount rows per image
    constexpr bool SPLIT = (AKIND == A_PLANES);                               // ... split from bytes by this kernel
    constexpr int IMGS = BM / 8;           // A_PLANES: images per tile

    // bit-plane mode pads the row stride: its 16-bit plane stores would otherwise hit the same bank eight times
    constexpr int AS_LD = SPLIT ? BM + 4 : BM;
    __shared__ __align__(16) uint32_t As[2][BKW][AS_LD];
    __shared__ __align__(16) uint32_t Bs[2][BKW][BN];
    __shared__ int32_t aux[(AKIND == A_CONV) ? 9 * BN : (SPLIT ? IMGS : 1)];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t rows_total = PLANES ? 8 * p.M : p.M;      // operand rows
    const int64_t tiles_m = (rows_total + BM - 1) / BM;
    const int64_t tile_m = blockIdx.x % tiles_m, tile_n = blockIdx.x / tiles_m;
    const int64_t m0 = tile_m * BM, n0 = tile_n * BN;       // m0 in operand rows
    const int64_t Kw = (p.K + 31) >> 5;
    const int64_t nchunks = (Kw + BKW - 1) / BKW;
    const uint32_t tail_mask = (p.K & 31) ? ((1u << (p.K & 31)) - 1u) : 0xffffffffu;

    // ---- loader roles: one A item per thread, (2*BN)/NT B items per thread
    const bool a_thread = tid < A_THREADS;
    const int a_row = tid % BM, a_half = (tid / BM) & 1;    // A_PACKED / A_CONV: row and which 4 of the 8 words
    const int a_img = (tid >> 4) % IMGS, a_seg = tid & 15;  // A_PLANES: image in tile and 16-byte segment of the chunk
    const int64_t am = SPLIT ? (m0 >> 3) + a_img : m0 + a_row;
    const bool a_ok = a_thread && am < (SPLIT ? p.M : rows_total);
    int pix_y = 0, pix_x = 0;
    int64_t pix_b = 0;
    if (AKIND == A_CONV && a_ok) {
        int64_t idx = am;
        int q = 0;
        int Wd = p.W, Hd = p.H;
        if (p.pool) { q = (int)(idx & 3); idx >>= 2; Wd >>= 1; Hd >>= 1; }
        pix_x = (int)(idx % Wd);
        idx /= Wd;
        pix_y = (int)(idx % Hd);
        pix_b = idx / Hd;
        if (p.pool) { pix_y = 2 * pix_y + (q >> 1); pix_x = 2 * pix_x + (q & 1); }
    }
    const bool a_vec = (AKIND == A_CONV) ? ((p.Cw & 3) == 0) : true;
    const bool b_vec = (AKIND == A_CONV) ? ((p.Cw & 3) == 0) : true;
    int32_t x_sum = 0;   // A_PLANES: running sum of this loader's bytes

    constexpr int B_ITEMS = (2 * BN) / NT;
    uint4 ra;
    uint4 rb[B_ITEMS];

    auto load_chunk = [&](int64_t c) {
        if (AKIND == A_PACKED || AKIND == A_PLANES_PRE) {
            ra = load_row_words(p.A + am * p.lda, a_ok, c * BKW + 4 * a_half, Kw, tail_mask, a_vec);
        } else if (AKIND == A_CONV) {
            ra = make_uint4(0u, 0u, 0u, 0u);
            const int64_t kw = c * BKW + 4 * a_half;
            if (a_ok && kw < Kw) {
                if (a_vec) {
                    const int tap = (int)(kw / p.Cw), cw = (int)(kw % p.Cw);
                    const int yy = pix_y + tap / 3 - 1, xx = pix_x + tap % 3 - 1;
                    if (yy >= 0 && yy < p.H && xx >= 0 && xx < p.W)
                        ra = *reinterpret_cast<const uint4 *>(p.A + ((pix_b * p.H + yy) * p.W + xx) * p.Cw + cw);
                } else {
                    uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (kw + i < Kw) {
                            const int tap = (int)((kw + i) / p.Cw), cw = (int)((kw + i) % p.Cw);
                            const int yy = pix_y + tap / 3 - 1, xx = pix_x + tap % 3 - 1;
                            if (yy >= 0 && yy < p.H && xx >= 0 && xx < p.W)
                                w[i] = p.A[((pix_b * p.H + yy) * p.W + xx) * p.Cw + cw];
                        }
                    }
                    ra = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        } else {   // A_PLANES: 16 bytes (inputs 256c + 16*seg ...) of image `am`
            ra = make_uint4(0u, 0u, 0u, 0u);
            const int64_t k0 = c * (32 * BKW) + 16 * a_seg;
            if (a_ok && k0 < p.K) {
                const uint8_t *src = p.X + am * p.ldx + k0;
                if (k0 + 16 <= p.K && ((reinterpret_cast<uintptr_t>(src) & 15u) == 0)) {
                    ra = *reinterpret_cast<const uint4 *>(src);
                } else {
                    uint32_t w[4] = {0u, 0u, 0u, 0u};
                    for (int i = 0; i < 16; ++i)
                        if (k0 + i < p.K) w[i >> 2] |= (uint32_t)src[i] << (8 * (i & 3));
                    ra = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        }
#pragma unroll
        for (int it = 0; it < B_ITEMS; ++it) {
            const int idx = tid + it * NT;
            const int b_row = idx % BN, b_half = idx / BN;
            const int64_t bn = n0 + b_row;
            rb[it] = load_row_words(p.B + bn * p.ldb, bn < p.N, c * BKW + 4 * b_half, Kw, tail_mask, b_vec);
        }
    };

    auto store_chunk = [&](int buf) {
        if (!a_thread) {
        } else if (SPLIT) {
            const uint32_t w[4] = {ra.x, ra.y, ra.z, ra.w};
            x_sum += (int32_t)(__vsadu4(ra.x, 0u) + __vsadu4(ra.y, 0u) + __vsadu4(ra.z, 0u) + __vsadu4(ra.w, 0u));
#pragma unroll
            for (int pl = 0; pl < 8; ++pl) {
                const uint32_t h = plane_nibble(w[0], pl) | (plane_nibble(w[1], pl) << 4) |
                                   (plane_nibble(w[2], pl) << 8) | (plane_nibble(w[3], pl) << 12);
                reinterpret_cast<uint16_t *>(&As[buf][a_seg >> 1][8 * a_img + pl])[a_seg & 1] = (uint16_t)h;
            }
        } else {
            As[buf][4 * a_half + 0][a_row] = ra.x;
            As[buf][4 * a_half + 1][a_row] = ra.y;
            As[buf][4 * a_half + 2][a_row] = ra.z;
            As[buf][4 * a_half + 3][a_row] = ra.w;
        }
#pragma unroll
        for (int it = 0; it < B_ITEMS; ++it) {
            const int idx = tid + it * NT;
            const int b_row = idx % BN, b_half = idx / BN;
            Bs[buf][4 * b_half + 0][b_row] = rb[it].x;
            Bs[buf][4 * b_half + 1][b_row] = rb[it].y;
            Bs[buf][4 * b_half + 2][b_row] = rb[it].z;
            Bs[buf][4 * b_half + 3][b_row] = rb[it].w;
        }
    };

    // ---- prologues
    if (AKIND == A_CONV) {   // popcount of every filter's weights per tap (correction for skipped taps)
        for (int e = tid; e < 9 * BN; e += NT) {
            const int tap = e / BN, col = e % BN;
            int32_t s = 0;
            if (n0 + col < p.N) {
                const uint32_t *wrow = p.B + (n0 + col) * p.ldb + (int64_t)tap * p.Cw;
                for (int cw = 0; cw < p.Cw; ++cw) s += __popc(wrow[cw]);
            }
            aux[e] = s;
        }
    }
    if (SPLIT) {
        if (tid < IMGS) aux[tid] = 0;
    }

    uint32_t acc[TM][TN];
    uint32_t ones[CSA ? TM : 1][CSA ? TN : 1];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0u;
    if (CSA) {
#pragma unroll
        for (int i = 0; i < (CSA ? TM : 1); ++i)
#pragma unroll
            for (int j = 0; j < (CSA ? TN : 1); ++j) ones[i][j] = 0u;
    }

    const int wr = warp * TM;
    const uint32_t one = p.one;
    if (nchunks > 0) {
        load_chunk(0);
        store_chunk(0);
    }
    __syncthreads();

    for (int64_t c = 0; c < nchunks; ++c) {
        const int buf = (int)(c & 1);
        if (c + 1 < nchunks) load_chunk(c + 1);
        // words of this chunk that can be non-zero (rounded up to a pair); the rest of the chunk is skipped
        const int kw_lim = (int)min((int64_t)BKW, ((Kw - c * BKW) + 1) & ~int64_t(1));

        if (!CSA) {
#pragma unroll
            for (int kw = 0; kw < BKW; ++kw) {
                if (kw < kw_lim) {
                    uint32_t a[TM], b[TN];
#pragma unroll
                    for (int q = 0; q < TM / 4; ++q) {
                        const uint4 v = *reinterpret_cast<const uint4 *>(&As[buf][kw][wr + 4 * q]);
                        a[4 * q] = v.x; a[4 * q + 1] = v.y; a[4 * q + 2] = v.z; a[4 * q + 3] = v.w;
                    }
#pragma unroll
                    for (int j = 0; j < TN; ++j) b[j] = Bs[buf][kw][lane + 32 * j];
#pragma unroll
                    for (int i = 0; i < TM; ++i)
#pragma unroll
                        for (int j = 0; j < TN; ++j)
                            acc[i][j] += (uint32_t)__popc(PLANES ? (a[i] & b[j]) : (a[i] ^ b[j]));
                }
            }
        } else {
#pragma unroll
            for (int kw = 0; kw < BKW; kw += 2) {
                if (kw < kw_lim) {
                    uint32_t b0[TN], b1[TN];
#pragma unroll
                    for (int j = 0; j < TN; ++j) { b0[j] = Bs[buf][kw][lane + 32 * j]; b1[j] = Bs[buf][kw + 1][lane + 32 * j]; }
#pragma unroll
                    for (int q = 0; q < TM / 4; ++q) {
                        const uint4 v0 = *reinterpret_cast<const uint4 *>(&As[buf][kw][wr + 4 * q]);
                        const uint4 v1 = *reinterpret_cast<const uint4 *>(&As[buf][kw + 1][wr + 4 * q]);
                        const uint32_t a0[4] = {v0.x, v0.y, v0.z, v0.w};
                        const uint32_t a1[4] = {v1.x, v1.y, v1.z, v1.w};
#pragma unroll
                        for (int ii = 0; ii < 4; ++ii)
#pragma unroll
                            for (int j = 0; j < TN; ++j) {
                                const int i = 4 * q + ii;
                                const uint32_t x0 = PLANES ? (a0[ii] & b0[j]) : (a0[ii] ^ b0[j]);
                                const uint32_t x1 = PLANES ? (a1[ii] & b1[j]) : (a1[ii] ^ b1[j]);
                                const uint32_t o = ones[CSA ? i : 0][CSA ? j : 0];
                                ones[CSA ? i : 0][CSA ? j : 0] = lop3_xor3(o, x0, x1);
                                acc[i][j] = (uint32_t)__popc(lop3_maj(o, x0, x1)) * one + acc[i][j];
                            }
                    }
                }
            }
        }

        if (c + 1 < nchunks) store_chunk(buf ^ 1);
        __syncthreads();
    }

    if (SPLIT) {
        if (a_thread) atomicAdd(&aux[a_img], x_sum);
        __syncthreads();
    }

    // ---- epilogue: integer result per output, then optional int32 store and optional Sign + repack
    int32_t thr_r[TN];
    uint32_t flip_r[TN];
#pragma unroll
    for (int j = 0; j < TN; ++j) {
        const int64_t col = n0 + lane + 32 * j;
        thr_r[j] = (p.out && col < p.N) ? p.thr[col] : 0;
        flip_r[j] = (p.out && p.flip && col < p.N) ? ((p.flip[col >> 5] >> (col & 31)) & 1u) : 0u;
    }
    // total popcount of output (i, j)
    auto total = [&](int i, int j) -> int32_t {
        int32_t P = (int32_t)acc[i][j];
        if (CSA) P = 2 * P + __popc(ones[CSA ? i : 0][CSA ? j : 0]);
        return P;
    };
    uint32_t keep = 0u;   // packed word this lane will store

    if (PLANES) {
        // this thread holds the 8 plane rows of TM/8 images: rows wr + 8*mi + pl
        constexpr int IPT = TM / 8;
#pragma unroll
        for (int mi = 0; mi < IPT; ++mi) {
            const int64_t img = (m0 >> 3) + IPT * warp + mi;
            const int32_t xs = SPLIT ? aux[IPT * warp + mi] : ((img < p.M) ? p.xsum[img] : 0);
#pragma unroll
            for (int j = 0; j < TN; ++j) {
                const int64_t col = n0 + lane + 32 * j;
                int32_t wsum = 0;
#pragma unroll
                for (int pl = 0; pl < 8; ++pl) wsum += total(8 * mi + pl, j) << pl;
                const int32_t dot = 2 * wsum - xs;
                const bool in = img < p.M && col < p.N;
                if (p.C && in) p.C[img * p.ldc + col] = dot;
                if (p.out) {
                    const bool bit = in && ((((uint32_t)(dot >= thr_r[j])) ^ flip_r[j]) & 1u);
                    const uint32_t word = __ballot_sync(0xffffffffu, bit);
                    if (lane == mi * TN + j) keep = word;
                }
            }
        }
        if (p.out && lane < IPT * TN) {
            const int64_t img = (m0 >> 3) + IPT * warp + (lane >> 2);
            const int64_t ow = (n0 >> 5) + (lane & 3);
            if (img < p.M && ow * 32 < p.N) p.out[img * p.ldo + ow] = keep;
        }
    } else {
        int32_t pooled[TN];
        uint32_t pooled_bit[TN];
        const bool pooled_mode = (AKIND == A_CONV) && p.pool;
#pragma unroll
        for (int i = 0; i < TM; ++i) {
            const int64_t row = m0 + wr + i;
            int32_t base = (int32_t)p.K;
            int inval = 0;     // A_CONV: bit t set if tap t falls outside the image
            if (AKIND == A_CONV) {
                int64_t idx = row < p.M ? row : 0;
                int q = 0, Wd = p.W, Hd = p.H;
                if (p.pool) { q = (int)(idx & 3); idx >>= 2; Wd >>= 1; Hd >>= 1; }
                int x = (int)(idx % Wd);
                int y = (int)((idx / Wd) % Hd);
                if (p.pool) { y = 2 * y + (q >> 1); x = 2 * x + (q & 1); }
                if (y == 0) inval |= 0x007;
                if (y == p.H - 1) inval |= 0x1c0;
                if (x == 0) inval |= 0x049;
                if (x == p.W - 1) inval |= 0x124;
                base = (int32_t)(p.Cw * 32) * (9 - __popc(inval));
            }
#pragma unroll
            for (int j = 0; j < TN; ++j) {
                const int64_t col = n0 + lane + 32 * j;
                int32_t P = total(i, j);
                if (AKIND == A_CONV && inval) {
                    for (int t = 0; t < 9; ++t)
                        if ((inval >> t) & 1) P -= aux[t * BN + lane + 32 * j];
                }
                const int32_t dot = base - 2 * P;
                const bool in = row < p.M && col < p.N;
                const bool q = in && (dot >= thr_r[j]);
                if (pooled_mode) {
                    // rows 4w..4w+3 of a thread are one pooling window
                    if ((i & 3) == 0) { pooled[j] = dot; pooled_bit[j] = q; }
                    else { pooled[j] = max(pooled[j], dot); pooled_bit[j] |= (uint32_t)q; }
                    if ((i & 3) == 3) {
                        if (p.C && in) p.C[(row >> 2) * p.ldc + col] = pooled[j];
                        if (p.out) {
                            const bool bit = in && ((pooled_bit[j] ^ flip_r[j]) & 1u);
                            const uint32_t word = __ballot_sync(0xffffffffu, bit);
                            if (lane == (((i >> 2) * TN + j) & 31)) keep = word;
                        }
                    }
                } else {
                    if (p.C && in) p.C[row * p.ldc + col] = dot;
                    if (p.out) {
                        const bool bit = in && (((uint32_t)q ^ flip_r[j]) & 1u);
                        const uint32_t word = __ballot_sync(0xffffffffu, bit);
                        if (lane == ((i * TN + j) & 31)) keep = word;
                    }
                }
            }
            // flush the 32 words gathered over the last 8 rows (or the 16 words of 4 pooled windows)
            if (p.out) {
                if (!pooled_mode && (i & 7) == 7) {
                    const int ri = (i & ~7) + (lane >> 2), j = lane & 3;
                    const int64_t orow = m0 + wr + ri;
                    const int64_t ow = (n0 >> 5) + j;
                    if (orow < p.M && ow * 32 < p.N) p.out[orow * p.ldo + ow] = keep;
                }
                if (pooled_mode && i == TM - 1 && lane < TM) {
                    const int wi = lane >> 2, j = lane & 3;
                    const int64_t orow = ((m0 + wr) >> 2) + wi;
                    const int64_t ow = (n0 >> 5) + j;
                    if (orow * 4 < p.M && ow * 32 < p.N) p.out[orow * p.ldo + ow] = keep;
                }
            }
        }
    }

    // padding words of the packed output (beyond ceil(N/32)) are written as 0 by the last column tile
    if (p.out && n0 + BN >= p.N) {
        const int64_t first_pad = (p.N + 31) >> 5;
        const int64_t npad = p.ldo - first_pad;
        if (npad > 0) {
            const bool pooled_mode = (AKIND == A_CONV) && p.pool;
            const int sh = PLANES ? 3 : (pooled_mode ? 2 : 0);   // operand rows per output row, log2
            const int64_t rows_out = pooled_mode ? (p.M >> 2) : p.M;
            const int64_t r0 = m0 >> sh;
            const int64_t nrows = BM >> sh;
            for (int64_t e = tid; e < nrows * npad; e += NT) {
                const int64_t r = r0 + e / npad;
                if (r < rows_out) p.out[r * p.ldo + first_pad + e % npad] = 0u;
            }
        }
    }
}

}  // namespace bnn_tile
