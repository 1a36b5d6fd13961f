// Stand-alone probe: how fast does one SM execute tcgen05.mma kind::i8 (M=128, N=256, K=32) when both operands
// already sit in shared memory and nothing is loaded?  One CTA per SM; one thread issues MMAS instructions in groups of
// four with a commit per group (the pattern of the library's main loop) and waits for the last group; cycles are read
// with clock64.  Also times the same with N=128.  Every wait is bounded.
// Build:  nvcc -gencode arch=compute_100a,code=sm_100a -O3 -o umma_i8_rate umma_i8_rate.cu
// Run:    ./umma_i8_rate
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#define CK(x) do{cudaError_t e=(x); if(e!=cudaSuccess){printf("CUDA error %s at %d\n",cudaGetErrorString(e),__LINE__); return 1;}}while(0)

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint64_t desc_sw128(uint32_t addr) {
    return (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ bool wait_parity(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < (1u << 22); ++i) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}

template <int N>
__global__ void __launch_bounds__(128, 1) k_rate(long long *cycles, int *status, int groups) {
    extern __shared__ uint8_t raw[];
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t tmem_base;
    for (int i = threadIdx.x; i < (128 + N) * 128 / 4; i += blockDim.x) reinterpret_cast<uint32_t *>(tiles)[i] = 0x01ff01ffu * (i | 1);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar)) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base)), "r"(256) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // generic-proxy writes of the tiles -> async proxy (MMA) reads
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tm = tmem_base;
    if (threadIdx.x == 0) {
        const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        const uint64_t a = desc_sw128(smem_u32(tiles)), b = desc_sw128(smem_u32(tiles + 128 * 128));
        const long long t0 = clock64();
        for (int g = 0; g < groups; ++g) {
#pragma unroll
            for (int k = 0; k < 4; ++k)
                asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
                             ::"r"(tm), "l"(a + 2 * k), "l"(b + 2 * k), "r"(idesc), "r"((g | k) ? 1u : 0u) : "memory");
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&bar)) : "memory");
        const bool ok = wait_parity(smem_u32(&bar), 0);
        const long long t1 = clock64();
        cycles[blockIdx.x] = t1 - t0;
        if (!ok) atomicExch(status, 1);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tm), "r"(256) : "memory");
    }
}

template <int N>
int run(int sms, int groups) {
    long long *cyc; int *status;
    CK(cudaMalloc(&cyc, sizeof(long long) * sms)); CK(cudaMalloc(&status, sizeof(int))); CK(cudaMemset(status, 0, sizeof(int)));
    const size_t smem = (128 + N) * 128 + 1024;
    CK(cudaFuncSetAttribute(k_rate<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
    k_rate<N><<<sms, 128, smem>>>(cyc, status, groups); CK(cudaDeviceSynchronize());
    cudaEventRecord(e0); k_rate<N><<<sms, 128, smem>>>(cyc, status, groups); cudaEventRecord(e1); CK(cudaDeviceSynchronize());
    float ms; cudaEventElapsedTime(&ms, e0, e1);
    long long h[1024]; int st; CK(cudaMemcpy(h, cyc, sizeof(long long) * sms, cudaMemcpyDeviceToHost)); CK(cudaMemcpy(&st, status, 4, cudaMemcpyDeviceToHost));
    double avg = 0, mx = 0; for (int i = 0; i < sms; ++i) { avg += h[i]; if (h[i] > mx) mx = h[i]; } avg /= sms;
    const double macs = 4.0 * groups * 128.0 * N * 32.0;
    printf("N=%d: %d MMA groups per SM, cycles avg %.0f max %.0f -> %.0f MAC/clk/SM; all %d SMs in %.3f ms -> %.0f int8 TOPS; wait %s\n",
           N, groups, avg, mx, macs / avg, sms, ms, 2.0 * macs * sms / (ms * 1e-3) / 1e12, st ? "GAVE UP" : "ok");
    cudaFree(cyc); cudaFree(status);
    return 0;
}

int main() {
    cudaDeviceProp p; CK(cudaGetDeviceProperties(&p, 0));
    printf("device %s, %d SMs\n", p.name, p.multiProcessorCount);
    for (int groups : {256, 4096}) { if (run<256>(p.multiProcessorCount, groups)) return 1; if (run<128>(p.multiProcessorCount, groups)) return 1; }
    return 0;
}
