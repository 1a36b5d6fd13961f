// Stand-alone probe: how fast does TMA bring L2-resident operand tiles into shared memory, per SM?
// `ctas` CTAs (one per SM, 200 KB of shared memory each) run P producer threads in different warps.  Every producer
// owns a ring of D stages of `ops` boxes of `rows` x `width` bytes and loads them (2-D, 128- or 64-byte swizzle, one
// barrier per stage) from a byte matrix of 32 MB that stays in L2, waiting for a stage's previous loads before it is
// reused, `iters` stages each.
// Printed per configuration: bytes and box rows per clock and SM (slowest CTA), the chip-wide TB/s at 1.65 GHz, and from a
// separate run with clock64 stamps what one iteration costs CTA 0's first producer (wait, expect_tx, the loads).
// Every wait is bounded; a wait that runs out sets the status word and ends the CTA's loop.
// Build:  nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -o tma_load_rate tma_load_rate.cu
// Run:    ./tma_load_rate
#include <cstdio>
#include <cstdint>
#include <cuda.h>
#include <cuda_runtime.h>
#define CK(x) do{cudaError_t e=(x); if(e!=cudaSuccess){printf("CUDA error %s at %d\n",cudaGetErrorString(e),__LINE__); return 1;}}while(0)
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool wait_parity(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < (1u << 22); ++i) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}
constexpr int MAXP = 4, MAXD = 16;
// rows x width bytes per box; the matrix has `mat_rows` rows of 4096 bytes
template <bool STAMP>
__global__ void __launch_bounds__(128, 1)
k_probe(const __grid_constant__ CUtensorMap map, long long *clocks, int *status, int P, int D, int rows, int width, int iters, int mat_rows,
        int ops, long long *stamps) {
    extern __shared__ uint8_t raw[];
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    __shared__ __align__(8) uint64_t bars[MAXP][MAXD];
    if (threadIdx.x == 0) {
        for (int p = 0; p < MAXP; ++p)
            for (int d = 0; d < MAXD; ++d) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bars[p][d])) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    long long t0 = clock64();
    if (lane == 0 && warp < P) {
        const uint32_t box_bytes = (uint32_t)(rows * width);      // `ops` boxes per stage, one barrier per stage
        uint8_t *mine = tiles + (size_t)warp * D * box_bytes * ops;
        const bool stamp = STAMP && blockIdx.x == 0 && warp == 0;
        int d = 0; uint32_t use = 0;                  // ring slot and how often it has been used before
        bool ok = true;
        uint32_t x = (uint32_t)((blockIdx.x * 7 + warp * 3) % (4096 / width)) * (uint32_t)width;
        uint32_t y = (uint32_t)((blockIdx.x * 131 + warp * 977) % (mat_rows / rows)) * (uint32_t)rows;
        for (int it = 0; it < iters && ok; ++it) {
            const uint32_t bar = smem_u32(&bars[warp][d]);
            const long long s0 = stamp ? clock64() : 0;
            if (use > 0 && !wait_parity(bar, (use - 1) & 1)) { atomicExch(status, 1); ok = false; break; }
            const long long s1 = stamp ? clock64() : 0;
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(box_bytes * ops) : "memory");
            const long long s2 = stamp ? clock64() : 0;
            for (int o = 0; o < ops; ++o) {
                asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                             ::"r"(smem_u32(mine + (uint32_t)(d * ops + o) * box_bytes)), "l"(&map), "r"((int)x), "r"((int)y), "r"(bar) : "memory");
                x += (uint32_t)width; if (x >= 4096u) { x = 0; y += (uint32_t)rows; if (y + rows > (uint32_t)mat_rows) y = 0; }
            }
            const long long s3 = stamp ? clock64() : 0;
            if (stamp && it >= 64 && it < 72) { long long *q = stamps + 4 * (it - 64); q[0] = s0 - t0; q[1] = s1 - s0; q[2] = s2 - s1; q[3] = s3 - s2; }
            if (++d == D) { d = 0; ++use; }
        }
        // drain: the last D loads
        for (int it = (iters > D ? iters - D : 0); it < iters && ok; ++it)
            if (!wait_parity(smem_u32(&bars[warp][it % D]), (it / D) & 1)) { atomicExch(status, 2); ok = false; }
    }
    __syncthreads();
    if (threadIdx.x == 0) clocks[blockIdx.x] = clock64() - t0;
}

typedef CUresult (*encode_fn_t)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
int main() {
    const int mat_rows = 8192;                       // 8192 x 4096 bytes = 32 MB
    uint8_t *mat; long long *clocks; int *status;
    CK(cudaMalloc(&mat, (size_t)mat_rows * 4096));
    CK(cudaMemset(mat, 1, (size_t)mat_rows * 4096));
    CK(cudaMalloc(&clocks, 148 * sizeof(long long)));
    CK(cudaMalloc(&status, sizeof(int)));
    CK(cudaMemset(status, 0, sizeof(int)));
    void *fn = nullptr; cudaDriverEntryPointQueryResult q;
    CK(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
    if (!fn) { printf("no cuTensorMapEncodeTiled\n"); return 1; }
    encode_fn_t enc = reinterpret_cast<encode_fn_t>(fn);
    const size_t smem = 200 * 1024 + 1024;
    CK(cudaFuncSetAttribute(k_probe<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    CK(cudaFuncSetAttribute(k_probe<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int sms = 0; CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0));
    int khz = 0; CK(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, 0));
    printf("SMs %d, nominal clock %.0f MHz\n", sms, khz / 1e3);
    printf("%5s %3s %3s %5s %5s %3s | %9s %9s %9s | clocks of CTA 0's first producer in its 69th iteration\n", "ctas", "P", "D", "rows", "width",
           "ops", "B/clk/SM", "rows/clk", "TB/s@1.65");
    long long *stamps; CK(cudaMalloc(&stamps, 32 * sizeof(long long)));
    struct Cfg { int ctas, P, D, rows, width, ops; };
    const Cfg cfgs[] = {
        {148, 1, 4, 128, 128, 1}, {148, 1, 12, 128, 128, 1}, {148, 2, 6, 128, 128, 1}, {148, 4, 3, 128, 128, 1},
        {148, 1, 6, 256, 128, 1}, {148, 1, 12, 64, 128, 1},  {148, 1, 12, 128, 64, 1}, {148, 4, 6, 128, 64, 1},
        {148, 1, 6, 128, 128, 2}, {148, 1, 3, 128, 128, 4},  {148, 2, 3, 128, 128, 2}, {148, 1, 6, 64, 128, 4},
        {16, 1, 8, 128, 128, 1},  {16, 4, 3, 128, 128, 1},   {16, 1, 6, 128, 128, 2},  {16, 1, 3, 128, 128, 4},
    };
    long long h[148];
    for (const Cfg &c : cfgs) {
        if ((size_t)c.P * c.D * c.rows * c.width * c.ops > 200 * 1024 || c.P > MAXP || c.D > MAXD) { printf("skip\n"); continue; }
        CUtensorMap map;
        cuuint64_t dims[2] = {4096, (cuuint64_t)mat_rows};
        cuuint64_t strides[1] = {4096};
        cuuint32_t box[2] = {(cuuint32_t)c.width, (cuuint32_t)c.rows};
        cuuint32_t estr[2] = {1, 1};
        CUresult r = enc(&map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, mat, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         c.width == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { printf("encode failed %d\n", (int)r); return 1; }
        const int iters = 2000;
        // first run: warms L2 and takes the time stamps (reading the clock slows the stamped thread); second run: the rate
        for (int rep = 0; rep < 2; ++rep) {
            if (rep == 0) k_probe<true><<<c.ctas, 128, smem>>>(map, clocks, status, c.P, c.D, c.rows, c.width, iters, mat_rows, c.ops, stamps);
            else k_probe<false><<<c.ctas, 128, smem>>>(map, clocks, status, c.P, c.D, c.rows, c.width, iters, mat_rows, c.ops, stamps);
            CK(cudaGetLastError());
            CK(cudaDeviceSynchronize());
        }
        CK(cudaMemcpy(h, clocks, c.ctas * sizeof(long long), cudaMemcpyDeviceToHost));
        long long worst = 0;
        for (int i = 0; i < c.ctas; ++i) worst = h[i] > worst ? h[i] : worst;
        const double bytes = (double)c.P * iters * c.rows * c.width * c.ops;
        long long hs[32]; CK(cudaMemcpy(hs, stamps, sizeof(hs), cudaMemcpyDeviceToHost));
        printf("%5d %3d %3d %5d %5d %3d | %9.1f %9.3f %9.2f | wait %lld expect %lld issue %lld, next iteration +%lld\n", c.ctas, c.P, c.D, c.rows,
               c.width, c.ops, bytes / worst, (double)c.P * iters * c.ops * c.rows / worst, bytes / worst * c.ctas * 1.65e9 / 1e12, hs[17], hs[18],
               hs[19], hs[20] - hs[16]);
    }
    int st = 0; CK(cudaMemcpy(&st, status, sizeof(int), cudaMemcpyDeviceToHost));
    printf("status %d (0 = no wait ran out)\n", st);
    return 0;
}
