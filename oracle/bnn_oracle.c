/*
 * CPU oracle for the run-time path of a Binarized Neural Network.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is the plain definition of
 * every quantity the GPU library computes, written on UNPACKED values (+1/-1 as
 * int8, inputs as uint8) with ordinary integer arithmetic: no bit packing, no
 * popcount, no XOR/XNOR identities, no folded thresholds derived from
 * BatchNorm, no tiling.  Only the tests, the smoke check and the CPU-baseline leg
 * of the benchmark may call it.  It shares no source, header, table or helper with
 * the CUDA library.
 *
 * OpenMP is used only to spread independent output rows over host cores; every
 * output element is still one straight sum in the order written here.  All sums
 * are exact integers (|sum| <= 255*K < 2^31), so evaluation order cannot matter.
 * Floating point (BatchNorm) is IEEE double; the file must be compiled with
 * -ffp-contract=off so that no multiply-add is fused.
 *
 * Every function is pinned by the CPU test-suite against something other than
 * itself (closed forms, numpy / torch library routines, brute force in Python,
 * the paper's identities); no function here is "parity unpinned".
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>

/* Eq. 1: deterministic binarization.  Sign(x) = +1 if x >= 0, else -1.
 * (-0.0 >= 0 is true, so both zeros map to +1.) */
static inline int8_t sign_of_double(double x) { return (x >= 0.0) ? (int8_t)1 : (int8_t)-1; }

void oracle_sign_f32(const float *x, int8_t *out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = sign_of_double((double)x[i]);
}

void oracle_sign_i32(const int32_t *x, int8_t *out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = (x[i] >= 0) ? (int8_t)1 : (int8_t)-1;
}

/* Section 4: the binary kernel must return what an ordinary matrix product
 * returns when its inputs are restricted to -1/+1.  So the oracle IS the ordinary
 * product: C[m][n] = sum_k A[m][k] * B[k][n], A is M x K, B is K x N, row-major. */
void oracle_gemm(const int8_t *A, const int8_t *B, int32_t *C, int64_t M, int64_t N, int64_t K)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        int32_t *c = C + m * N;
        for (int64_t n = 0; n < N; ++n) c[n] = 0;
        for (int64_t k = 0; k < K; ++k) {
            const int32_t a = (int32_t)A[m * K + k];
            const int8_t *b = B + k * N;
            for (int64_t n = 0; n < N; ++n) c[n] += a * (int32_t)b[n];
        }
    }
}

/* Section 1.6, Eq. 6 (first line): s = x . w with x an 8-bit unsigned input
 * vector and w in {-1,+1}.  X is M x K (uint8), W is K x N (int8). */
void oracle_first_layer(const uint8_t *X, const int8_t *W, int32_t *S, int64_t M, int64_t N, int64_t K)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        int32_t *s = S + m * N;
        for (int64_t n = 0; n < N; ++n) s[n] = 0;
        for (int64_t k = 0; k < K; ++k) {
            const int32_t x = (int32_t)X[m * K + k];
            const int8_t *w = W + k * N;
            for (int64_t n = 0; n < N; ++n) s[n] += x * (int32_t)w[n];
        }
    }
}

/* Section 1.6, Eq. 7 and Algorithm 4 step 1, taken literally:
 * s = sum_{n=1..8} 2^(n-1) * (x^n . w), x^n in {0,1} the n-th bit of x (n=1 least
 * significant, n=8 most significant).  Kept as a separate routine so that the
 * bit-plane identity is itself tested (it must equal oracle_first_layer). */
void oracle_first_layer_bitplanes(const uint8_t *X, const int8_t *W, int32_t *S, int64_t M, int64_t N,
                                  int64_t K)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) {
            int32_t a1 = 0;
            for (int plane = 1; plane <= 8; ++plane) {
                int32_t dot = 0;
                for (int64_t k = 0; k < K; ++k) {
                    const int32_t xbit = ((int32_t)X[m * K + k] >> (plane - 1)) & 1;
                    dot += xbit * (int32_t)W[k * N + n];
                }
                a1 += (1 << (plane - 1)) * dot;
            }
            S[m * N + n] = a1;
        }
    }
}

/* Run-time BatchNorm of one pre-activation with stored statistics, in double:
 * y = gamma * ((x - mean) / sqrt(var + eps)) + beta.  The parameters are the
 * float32 values widened to double.  The operation order is part of the
 * definition: subtract, divide by the square root, multiply, add. */
static inline double batchnorm_f64(double x, float gamma, float beta, float mean, float var, double eps)
{
    const double xhat = (x - (double)mean) / sqrt((double)var + eps);
    return (double)gamma * xhat + (double)beta;
}

void oracle_batchnorm(const int32_t *S, const float *gamma, const float *beta, const float *mean,
                      const float *var, double eps, double *Y, int64_t M, int64_t N)
{
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n)
            Y[m * N + n] = batchnorm_f64((double)S[m * N + n], gamma[n], beta[n], mean[n], var[n], eps);
}

/* Algorithm 4, hidden layer: a^b = Sign(BatchNorm(s, theta)), per channel n. */
void oracle_sign_batchnorm(const int32_t *S, const float *gamma, const float *beta, const float *mean,
                           const float *var, double eps, int8_t *out, int64_t M, int64_t N)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n)
            out[m * N + n] =
                sign_of_double(batchnorm_f64((double)S[m * N + n], gamma[n], beta[n], mean[n], var[n], eps));
}

/* Hidden layer when the caller states the decision as an integer rule:
 * out = +1 iff (s >= thr[n]) differs from flip[n]  (flip[n] in {0,1}; flip may be NULL = all 0). */
void oracle_threshold(const int32_t *S, const int32_t *thr, const uint8_t *flip, int8_t *out, int64_t M,
                      int64_t N)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            const int ge = S[m * N + n] >= thr[n];
            const int f = flip ? (flip[n] != 0) : 0;
            out[m * N + n] = (ge != f) ? (int8_t)1 : (int8_t)-1;
        }
}

/* Section 3.3: apply each 3x3 filter on the map and accumulate the products.
 * act: B x H x W x Cin (NHWC, int8 +-1), wgt: Cout x 3 x 3 x Cin (int8 +-1),
 * out: B x H x W x Cout int32.  Stride 1, one pixel of padding on each side; a
 * tap that falls outside the image contributes 0 (it is skipped). */
void oracle_conv3x3(const int8_t *act, const int8_t *wgt, int32_t *out, int64_t B, int64_t H, int64_t W,
                    int64_t Cin, int64_t Cout)
{
#pragma omp parallel for schedule(static) collapse(2)
    for (int64_t b = 0; b < B; ++b)
        for (int64_t y = 0; y < H; ++y)
            for (int64_t x = 0; x < W; ++x)
                for (int64_t n = 0; n < Cout; ++n) {
                    int32_t s = 0;
                    for (int dy = -1; dy <= 1; ++dy)
                        for (int dx = -1; dx <= 1; ++dx) {
                            const int64_t yy = y + dy, xx = x + dx;
                            if (yy < 0 || yy >= H || xx < 0 || xx >= W) continue;
                            const int8_t *a = act + ((b * H + yy) * W + xx) * Cin;
                            const int8_t *w = wgt + ((n * 3 + (dy + 1)) * 3 + (dx + 1)) * Cin;
                            for (int64_t c = 0; c < Cin; ++c) s += (int32_t)a[c] * (int32_t)w[c];
                        }
                    out[((b * H + y) * W + x) * Cout + n] = s;
                }
}

/* The same convolution for the first layer, whose input is 8-bit unsigned. */
void oracle_conv3x3_u8(const uint8_t *act, const int8_t *wgt, int32_t *out, int64_t B, int64_t H, int64_t W,
                       int64_t Cin, int64_t Cout)
{
#pragma omp parallel for schedule(static) collapse(2)
    for (int64_t b = 0; b < B; ++b)
        for (int64_t y = 0; y < H; ++y)
            for (int64_t x = 0; x < W; ++x)
                for (int64_t n = 0; n < Cout; ++n) {
                    int32_t s = 0;
                    for (int dy = -1; dy <= 1; ++dy)
                        for (int dx = -1; dx <= 1; ++dx) {
                            const int64_t yy = y + dy, xx = x + dx;
                            if (yy < 0 || yy >= H || xx < 0 || xx >= W) continue;
                            const uint8_t *a = act + ((b * H + yy) * W + xx) * Cin;
                            const int8_t *w = wgt + ((n * 3 + (dy + 1)) * 3 + (dx + 1)) * Cin;
                            for (int64_t c = 0; c < Cin; ++c) s += (int32_t)a[c] * (int32_t)w[c];
                        }
                    out[((b * H + y) * W + x) * Cout + n] = s;
                }
}

/* 2x2 max-pooling with stride 2 on the integer sums (H and W even).
 * in: B x H x W x C int32, out: B x H/2 x W/2 x C int32. */
void oracle_maxpool2x2(const int32_t *in, int32_t *out, int64_t B, int64_t H, int64_t W, int64_t C)
{
    const int64_t Ho = H / 2, Wo = W / 2;
    for (int64_t b = 0; b < B; ++b)
        for (int64_t y = 0; y < Ho; ++y)
            for (int64_t x = 0; x < Wo; ++x)
                for (int64_t c = 0; c < C; ++c) {
                    int32_t best = in[((b * H + 2 * y) * W + 2 * x) * C + c];
                    for (int dy = 0; dy < 2; ++dy)
                        for (int dx = 0; dx < 2; ++dx) {
                            const int32_t v = in[((b * H + 2 * y + dy) * W + 2 * x + dx) * C + c];
                            if (v > best) best = v;
                        }
                    out[((b * Ho + y) * Wo + x) * C + c] = best;
                }
}
