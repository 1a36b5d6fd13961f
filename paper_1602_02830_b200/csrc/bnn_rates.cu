// bnn_measure_pipe_rates: the issue rates the popcount roofline is derived from, measured on the device the context is
// bound to, so that a benchmark can take its denominator from the same run instead of from a data sheet.
// Section 4 counts an XNOR-popcount step as "1 + 4 + 1" cycles on the GPUs of its time (xnor, popcount, accumulate);
// here the three instructions of Eq. 8 are timed in a register-only loop, alone and together.
#include "bnn_common.cuh"

namespace {

constexpr int RATE_ITERS = 2048;   // x 8 independent chains per thread

// MODE 0: popc only; 1: lop3 only; 2: the loop of Eq. 8 (xor, popc, add).  One CTA of 1024 threads per SM; thread 0
// of every CTA records the cycles its CTA needed (clock64 ticks at the SM clock).
template <int MODE>
__global__ void __launch_bounds__(1024) k_pipe_rate(uint32_t *sink, long long *cycles, uint32_t seed) {
    uint32_t a[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) a[i] = seed * (threadIdx.x + 1) * (i + 3);
    const uint32_t b = seed ^ 0x9e3779b9u, c = seed * 77u;
    __syncthreads();
    const long long t0 = clock64();
#pragma unroll 1
    for (int it = 0; it < RATE_ITERS; ++it) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (MODE == 0) {
                asm volatile("popc.b32 %0, %0;" : "+r"(a[i]));
            } else if (MODE == 1) {
                asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(a[i]) : "r"(b), "r"(c));
            } else {
                uint32_t t, q;
                asm volatile("xor.b32 %0, %1, %2;" : "=r"(t) : "r"(a[i]), "r"(b));
                asm volatile("popc.b32 %0, %1;" : "=r"(q) : "r"(t));
                asm volatile("add.u32 %0, %0, %1;" : "+r"(a[i]) : "r"(q));
            }
        }
    }
    __syncthreads();
    const long long t1 = clock64();
    uint32_t s = b ^ c;
#pragma unroll
    for (int i = 0; i < 8; ++i) s ^= a[i];
    sink[blockIdx.x * blockDim.x + threadIdx.x] = s;
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

}  // namespace

// scratch: device memory, at least sm_count * (1024 * 4 + 8) bytes, 8-byte aligned.  Synchronises the context's stream.
extern "C" int bnn_measure_pipe_rates(bnn_ctx *ctx, void *scratch, size_t scratch_bytes, double *popc_per_clk_per_sm,
                                      double *lop3_per_clk_per_sm, double *xor_popc_add_per_clk_per_sm) {
    if (!ctx || !scratch || !popc_per_clk_per_sm || !lop3_per_clk_per_sm || !xor_popc_add_per_clk_per_sm) return BNN_ERR_INVALID_ARG;
    const size_t need = (size_t)ctx->sm_count * (1024 * 4 + 8);
    if (scratch_bytes < need) return BNN_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(scratch) & 7u) return BNN_ERR_ALIGNMENT;
    bnn_device_guard guard(ctx);
    if (!guard.ok) return BNN_ERR_CUDA;
    long long *cycles = static_cast<long long *>(scratch);
    uint32_t *sink = reinterpret_cast<uint32_t *>(static_cast<char *>(scratch) + (size_t)ctx->sm_count * 8);
    double *out[3] = {popc_per_clk_per_sm, lop3_per_clk_per_sm, xor_popc_add_per_clk_per_sm};
    long long host[1024];
    if (ctx->sm_count > 1024) return BNN_ERR_INVALID_ARG;
    for (int mode = 0; mode < 3; ++mode) {
        for (int rep = 0; rep < 2; ++rep) {      // the first launch warms the instruction cache and the clocks
            if (mode == 0) k_pipe_rate<0><<<ctx->sm_count, 1024, 0, ctx->stream>>>(sink, cycles, 12345u + rep);
            else if (mode == 1) k_pipe_rate<1><<<ctx->sm_count, 1024, 0, ctx->stream>>>(sink, cycles, 12345u + rep);
            else k_pipe_rate<2><<<ctx->sm_count, 1024, 0, ctx->stream>>>(sink, cycles, 12345u + rep);
            if (int st = bnn_check_launch(ctx)) return st;
        }
        BNN_CUDA_TRY(ctx, cudaMemcpyAsync(host, cycles, sizeof(long long) * ctx->sm_count, cudaMemcpyDeviceToHost, ctx->stream));
        BNN_CUDA_TRY(ctx, cudaStreamSynchronize(ctx->stream));
        double sum = 0.0;
        for (int i = 0; i < ctx->sm_count; ++i) sum += (double)host[i];
        const double avg = sum / ctx->sm_count;
        *out[mode] = avg > 0.0 ? 1024.0 * 8.0 * RATE_ITERS / avg : 0.0;   // thread-level results per clock and SM
    }
    return BNN_OK;
}
