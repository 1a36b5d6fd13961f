// Stand-alone probe: latency of tcgen05.ld 32x32b (tensor memory -> registers) with 1..16 warps loading at once.
// Modes: 0 one x16 load, 1 one x32 load, 2 two x32 loads back to back, 3 four x32 loads each waited for and used.
// Printed per warp of CTA 0: clocks until the load(s) were issued / until tcgen05.wait::ld returned.
// Build:  nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -o tmem_ld_latency tmem_ld_latency.cu
// Run:    ./tmem_ld_latency
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#define CK(x) do{cudaError_t e=(x); if(e!=cudaSuccess){printf("CUDA error %s at %d\n",cudaGetErrorString(e),__LINE__); return 1;}}while(0)
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
#define R8(r, o) "=r"(r[o+0]), "=r"(r[o+1]), "=r"(r[o+2]), "=r"(r[o+3]), "=r"(r[o+4]), "=r"(r[o+5]), "=r"(r[o+6]), "=r"(r[o+7])
__device__ __forceinline__ void ld16(uint32_t a, uint32_t (&r)[64], int o) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[o+0]), "=r"(r[o+1]), "=r"(r[o+2]), "=r"(r[o+3]), "=r"(r[o+4]), "=r"(r[o+5]), "=r"(r[o+6]), "=r"(r[o+7]),
          "=r"(r[o+8]), "=r"(r[o+9]), "=r"(r[o+10]), "=r"(r[o+11]), "=r"(r[o+12]), "=r"(r[o+13]), "=r"(r[o+14]), "=r"(r[o+15]) : "r"(a) : "memory");
}
__device__ __forceinline__ void ld32(uint32_t a, uint32_t (&r)[64], int o) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[o+0]), "=r"(r[o+1]), "=r"(r[o+2]), "=r"(r[o+3]), "=r"(r[o+4]), "=r"(r[o+5]), "=r"(r[o+6]), "=r"(r[o+7]),
          "=r"(r[o+8]), "=r"(r[o+9]), "=r"(r[o+10]), "=r"(r[o+11]), "=r"(r[o+12]), "=r"(r[o+13]), "=r"(r[o+14]), "=r"(r[o+15]),
          "=r"(r[o+16]), "=r"(r[o+17]), "=r"(r[o+18]), "=r"(r[o+19]), "=r"(r[o+20]), "=r"(r[o+21]), "=r"(r[o+22]), "=r"(r[o+23]),
          "=r"(r[o+24]), "=r"(r[o+25]), "=r"(r[o+26]), "=r"(r[o+27]), "=r"(r[o+28]), "=r"(r[o+29]), "=r"(r[o+30]), "=r"(r[o+31]) : "r"(a) : "memory");
}
__device__ __forceinline__ void ldwait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// mode 0: one x16; 1: one x32; 2: two x32 back to back (64 columns); 3: four x32 in sequence each waited (loop of 4)
template <int MODE>
__global__ void __launch_bounds__(512, 1) k_ld(long long *out, uint32_t *sink, int active_warps) {
    __shared__ uint32_t tmem_base;
    const int warp = threadIdx.x >> 5;
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tm = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)((warp >> 2) * 64);
    uint32_t r[64];
    for (int i = 0; i < 64; ++i) r[i] = 0;
    uint32_t acc = 0;
    long long t0 = 0, t1 = 0, t2 = 0;
    __syncthreads();
    if (warp < active_warps) {
        for (int rep = 0; rep < 4; ++rep) {      // the last repetition is reported
            t0 = clock64();
            if (MODE == 0) { ld16(tm, r, 0); t1 = clock64(); ldwait(); }
            if (MODE == 1) { ld32(tm, r, 0); t1 = clock64(); ldwait(); }
            if (MODE == 2) { ld32(tm, r, 0); ld32(tm + 32, r, 32); t1 = clock64(); ldwait(); }
            if (MODE == 3) { for (int c = 0; c < 4; ++c) { ld32(tm + 16 * (c & 1), r, 0); ldwait(); acc += r[5]; } t1 = clock64(); }
            t2 = clock64();
            for (int i = 0; i < 64; ++i) acc += r[i];
        }
        if (blockIdx.x == 0 && (threadIdx.x & 31) == 0) { out[warp * 2] = t1 - t0; out[warp * 2 + 1] = t2 - t0; }
    }
    sink[blockIdx.x * blockDim.x + threadIdx.x] = acc;
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
    }
}
template <int MODE> int run(int aw) {
    long long *out; uint32_t *sink;
    CK(cudaMalloc(&out, 32 * 8)); CK(cudaMalloc(&sink, 148 * 512 * 4)); CK(cudaMemset(out, 0, 32 * 8));
    k_ld<MODE><<<148, 512>>>(out, sink, aw); CK(cudaDeviceSynchronize());
    long long h[32]; CK(cudaMemcpy(h, out, sizeof(h), cudaMemcpyDeviceToHost));
    printf("mode %d, %2d warps: issue/total clk per warp:", MODE, aw);
    for (int w = 0; w < aw; ++w) printf(" %lld/%lld", h[2 * w], h[2 * w + 1]);
    printf("\n");
    cudaFree(out); cudaFree(sink);
    return 0;
}
int main() {
    for (int aw : {1, 4, 8, 16}) { if (run<0>(aw)) return 1; if (run<1>(aw)) return 1; if (run<2>(aw)) return 1; if (run<3>(aw)) return 1; }
    return 0;
}
