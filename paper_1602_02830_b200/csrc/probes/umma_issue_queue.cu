// Stand-alone probe: what does issuing tcgen05.mma cost the issuing thread, and do two issuing warps overlap?
// One CTA per SM, operands resident in shared memory (nothing is loaded), kind::mxf4.block_scale M=128 N=192 K=64 with
// unit scale factors (the library's 4-bit configuration).  Thread 0 (and, with mode bit 16, thread 32 into a second
// accumulator) issues 12 groups of four MMAs and stamps clock64 after every group.  Mode bits add work per group:
//   1  tcgen05.commit to a barrier nobody waits on      2  a clock64 spin of `delay` clocks
//   4  try_wait on an already completed barrier + fence  8  __nanosleep(delay)      16  second issuing warp
// Printed: the stamps of CTA 0's first issuer and when its last group completed.  Every wait is bounded.
// Build:  nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -o umma_issue_queue umma_issue_queue.cu
// Run:    ./umma_issue_queue
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
constexpr int NM = 48;
template <int N, bool F4>
__global__ void __launch_bounds__(128, 1) k_probe(long long *stamps, int *status, int mode, int delay) {
    extern __shared__ uint8_t raw[];
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    __shared__ __align__(8) uint64_t bar, bar2, bar3, barB;
    __shared__ long long t_end[2];
    __shared__ uint32_t tmem_base;
    for (int i = threadIdx.x; i < (128 + N) * 128 / 4; i += blockDim.x) reinterpret_cast<uint32_t *>(tiles)[i] = F4 ? 0x2a2a2a2au : 0x01ff01ffu;
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar)) : "memory");
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar2)) : "memory");
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&barB)) : "memory");
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar3)) : "memory");
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&bar3)) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tm = tmem_base, sf = tm + 480;
    {
        const int q = threadIdx.x >> 5;
        const uint32_t v = 0x7f7f7f7fu;
        asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1};"
                     ::"r"(sf + ((uint32_t)(32 * q) << 16)), "r"(v) : "memory");
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const bool second = (threadIdx.x == 32) && (mode & 16);
    if (threadIdx.x == 0 || second) {
        const uint32_t tmd = second ? tm + 192 : tm;
        const uint32_t mybar = second ? smem_u32(&barB) : smem_u32(&bar);
        const uint32_t idesc4 = (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | (1u << 23) | ((uint32_t)(128 >> 4) << 24);
        const uint32_t idesc8 = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        const uint64_t a = desc_sw128(smem_u32(tiles)), b = desc_sw128(smem_u32(tiles + 128 * 128));
        long long st[NM + 2];
        st[0] = clock64();
#pragma unroll
        for (int i = 0; i < NM; ++i) {
            if (F4)
                asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                             "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
                             ::"r"(tmd), "l"(a + 2 * (i & 3)), "l"(b + 2 * (i & 3)), "r"(idesc4), "r"(i ? 1u : 0u), "r"(sf), "r"(sf) : "memory");
            else
                asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                             "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
                             ::"r"(tmd), "l"(a + 2 * (i & 3)), "l"(b + 2 * (i & 3)), "r"(idesc8), "r"(i ? 1u : 0u) : "memory");
            if ((i & 3) == 3) {
                if (mode & 1) asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&bar2)) : "memory");
                if (mode & 2) { const long long c = clock64(); while (clock64() - c < delay) {} }
                if (mode & 4) { wait_parity(smem_u32(&bar3), 0); asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
                if (mode & 8) __nanosleep(delay);
                st[i / 4 + 1] = clock64();
            }
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(mybar) : "memory");
        const bool ok = wait_parity(mybar, 0);
        st[NM + 1] = clock64();
        if (blockIdx.x == 0 && !second) for (int i = 0; i < NM + 2; ++i) stamps[i] = st[i] - st[0];
        if (!ok) atomicExch(status, 1);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tm), "r"(512) : "memory");
    }
}
template <int N, bool F4> int run(int sms, int mode, int delay) {
    long long *st; int *status;
    CK(cudaMalloc(&st, sizeof(long long) * (NM + 2))); CK(cudaMalloc(&status, 4)); CK(cudaMemset(status, 0, 4));
    const size_t smem = (128 + N) * 128 + 1024;
    CK(cudaFuncSetAttribute(k_probe<N, F4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    for (int r = 0; r < 2; ++r) { k_probe<N, F4><<<sms, 128, smem>>>(st, status, mode, delay); CK(cudaDeviceSynchronize()); }
    long long h[NM + 2]; int s;
    CK(cudaMemcpy(h, st, sizeof(h), cudaMemcpyDeviceToHost)); CK(cudaMemcpy(&s, status, 4, cudaMemcpyDeviceToHost));
    printf("mode %d delay %d N=%d %s status %d; clocks after each group:", mode, delay, N, F4 ? "mxf4" : "i8", s);
    for (int i = 1; i <= NM / 4; ++i) printf(" %lld", h[i]);
    printf(" | all done %lld\n", h[NM + 1]);
    return 0;
}
int main() {
    cudaDeviceProp p; CK(cudaGetDeviceProperties(&p, 0));
    const int sms = p.multiProcessorCount;
    int modes[][2] = {{1,0},{17,0},{5,0},{21,0},{3,150},{19,150},{3,300},{19,300},{3,500},{19,500}};
    for (auto &m : modes) if (run<192, true>(sms, m[0], m[1])) return 1;
    return 0;
}
