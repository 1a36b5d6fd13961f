// The comparison point of Section 4 / Fig. 3: a "quite unoptimized" matrix multiplication kernel that multiplies
// the +-1 values as ordinary 32-bit floats (one thread per output, no tiling, no shared memory).  It exists only so
// that the paper's speed ratios (XNOR kernel vs baseline kernel, vs cuBLAS) can be put next to B200 numbers; nothing
// in the library's own path calls it.
#include "bnn_common.cuh"

namespace {
__global__ void __launch_bounds__(256) k_baseline_f32(const float *__restrict__ A, const float *__restrict__ B,
                                                      float *__restrict__ C, int64_t M, int64_t N, int64_t K) {
    const int64_t n = (int64_t)blockIdx.x * 16 + (threadIdx.x & 15);
    const int64_t m = (int64_t)blockIdx.y * 16 + (threadIdx.x >> 4);
    if (m >= M || n >= N) return;
    float acc = 0.0f;
    for (int64_t k = 0; k < K; ++k) acc += A[m * K + k] * B[k * N + n];
    C[m * N + n] = acc;
}
}  // namespace

extern "C" int bnn_baseline_gemm_f32(bnn_ctx *ctx, const float *A, const float *B, float *C, int64_t M, int64_t N,
                                     int64_t K) {
    if (!ctx || M < 0 || N < 0 || K < 0) return BNN_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return BNN_OK;
    if (!A || !B || !C) return BNN_ERR_INVALID_ARG;
    if ((M + 15) / 16 > 65535) return BNN_ERR_INVALID_ARG;
    bnn_device_guard guard(ctx);
    if (!guard.ok) return BNN_ERR_CUDA;
    dim3 grid((unsigned)((N + 15) / 16), (unsigned)((M + 15) / 16));
    k_baseline_f32<<<grid, 256, 0, ctx->stream>>>(A, B, C, M, N, K);
    return bnn_check_launch(ctx);
}
