// Stand-alone probe of the sm_100a integer-pipe and legacy tensor-op issue rates that the library's
// roofline is derived from: POPC, LOP3, integer add, the xor+popc+add loop of Eq. 8, POPC with independent
// LOP3s beside it, and the legacy mma.sync b1 (xor.popc / and.popc) and s8 shapes.
// Build:  nvcc -gencode arch=compute_100a,code=sm_100a -O3 -o pipe_rates pipe_rates.cu
// Run:    ./pipe_rates            (one CTA per SM; cycles are read with clock64 inside the kernel)
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#define CK(x) do{cudaError_t e=(x); if(e!=cudaSuccess){printf("CUDA error %s at %d\n",cudaGetErrorString(e),__LINE__); return 1;}}while(0)

constexpr int ITERS = 4096;

template<int MODE>
__global__ void __launch_bounds__(1024) k_pipe(uint32_t* out, long long* cyc, uint32_t seed) {
  uint32_t a[8];
  #pragma unroll
  for (int i=0;i<8;i++) a[i] = seed*(threadIdx.x+1)*(i+3);
  uint32_t b = seed ^ 0x9e3779b9u, c = seed*77u;
  __syncthreads();
  long long t0 = clock64();
  #pragma unroll 1
  for (int it=0; it<ITERS; ++it) {
    #pragma unroll
    for (int i=0;i<8;i++) {
      if (MODE==0) { asm volatile("popc.b32 %0, %0;" : "+r"(a[i])); }
      else if (MODE==1) { asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(a[i]) : "r"(b), "r"(c)); }
      else if (MODE==2) { asm volatile("add.u32 %0, %0, %1;" : "+r"(a[i]) : "r"(b)); }
      else if (MODE==3) { // plain inner loop: xor, popc, add  (acc += popc(acc_prev ^ b)) -- dependent chain per i, 8 chains
        uint32_t t; asm volatile("xor.b32 %0, %1, %2;" : "=r"(t) : "r"(a[i]), "r"(b));
        uint32_t p; asm volatile("popc.b32 %0, %1;" : "=r"(p) : "r"(t));
        asm volatile("add.u32 %0, %0, %1;" : "+r"(a[i]) : "r"(p));
      }
      else if (MODE==4) { // fp32 fma for reference
        float f = __uint_as_float(a[i]); asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(f) : "f"(1.0001f), "f"(0.5f)); a[i]=__float_as_uint(f);
      }
      else if (MODE==5) { // popc + 2 independent lop3 : do they overlap?
        asm volatile("popc.b32 %0, %0;" : "+r"(a[i]));
        asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(b) : "r"(a[i]), "r"(c));
        asm volatile("lop3.b32 %0, %0, %1, %2, 0xe8;" : "+r"(c) : "r"(a[i]), "r"(b));
      }
      else if (MODE==6) { // popc + 4 lop3
        asm volatile("popc.b32 %0, %0;" : "+r"(a[i]));
        uint32_t &x = a[(i+1)&7], &y = a[(i+2)&7];
        asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(b) : "r"(x), "r"(c));
        asm volatile("lop3.b32 %0, %0, %1, %2, 0xe8;" : "+r"(c) : "r"(y), "r"(b));
        asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x) : "r"(b), "r"(c));
        asm volatile("lop3.b32 %0, %0, %1, %2, 0xe8;" : "+r"(y) : "r"(x), "r"(b));
      }
    }
  }
  long long t1 = clock64();
  uint32_t s=b^c; 
  #pragma unroll
  for (int i=0;i<8;i++) s ^= a[i];
  out[blockIdx.x*blockDim.x+threadIdx.x] = s;
  if (threadIdx.x==0) cyc[blockIdx.x] = t1-t0;
}

// legacy b1 mma: m16n8k256, per warp-instr 16*8*256 bit-MACs
template<int OP> // 0 xor, 1 and
__global__ void __launch_bounds__(1024) k_bmma(uint32_t* out, long long* cyc, uint32_t seed) {
  int acc[4][4];
  #pragma unroll
  for (int j=0;j<4;j++) for (int i=0;i<4;i++) acc[j][i]=0;
  uint32_t a0=seed*threadIdx.x, a1=a0*3, a2=a0*5, a3=a0*7, b0=a0*11, b1=a0*13;
  __syncthreads();
  long long t0 = clock64();
  #pragma unroll 1
  for (int it=0; it<ITERS; ++it) {
    #pragma unroll
    for (int j=0;j<4;j++) {
      if (OP==0)
      asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.xor.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(acc[j][0]),"+r"(acc[j][1]),"+r"(acc[j][2]),"+r"(acc[j][3]) : "r"(a0),"r"(a1),"r"(a2),"r"(a3),"r"(b0),"r"(b1));
      else
      asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.and.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(acc[j][0]),"+r"(acc[j][1]),"+r"(acc[j][2]),"+r"(acc[j][3]) : "r"(a0),"r"(a1),"r"(a2),"r"(a3),"r"(b0),"r"(b1));
    }
  }
  long long t1 = clock64();
  int s=0;
  #pragma unroll
  for (int j=0;j<4;j++) for (int i=0;i<4;i++) s^=acc[j][i];
  out[blockIdx.x*blockDim.x+threadIdx.x] = s;
  if (threadIdx.x==0) cyc[blockIdx.x] = t1-t0;
}

// legacy s8 mma m16n8k32: 16*8*32 MACs per warp instr
__global__ void __launch_bounds__(1024) k_imma(uint32_t* out, long long* cyc, uint32_t seed) {
  int acc[4][4];
  #pragma unroll
  for (int j=0;j<4;j++) for (int i=0;i<4;i++) acc[j][i]=0;
  uint32_t a0=seed*threadIdx.x, a1=a0*3, a2=a0*5, a3=a0*7, b0=a0*11, b1=a0*13;
  __syncthreads();
  long long t0 = clock64();
  #pragma unroll 1
  for (int it=0; it<ITERS; ++it) {
    #pragma unroll
    for (int j=0;j<4;j++)
      asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(acc[j][0]),"+r"(acc[j][1]),"+r"(acc[j][2]),"+r"(acc[j][3]) : "r"(a0),"r"(a1),"r"(a2),"r"(a3),"r"(b0),"r"(b1));
  }
  long long t1 = clock64();
  int s=0;
  #pragma unroll
  for (int j=0;j<4;j++) for (int i=0;i<4;i++) s^=acc[j][i];
  out[blockIdx.x*blockDim.x+threadIdx.x] = s;
  if (threadIdx.x==0) cyc[blockIdx.x] = t1-t0;
}

template<typename F>
int run(const char* name, F launch, int nblk, int threads, double per_thread_per_iter, double unit_scale, const char* unit) {
  uint32_t* out; long long* cyc;
  CK(cudaMalloc(&out, sizeof(uint32_t)*nblk*1024)); CK(cudaMalloc(&cyc, sizeof(long long)*nblk));
  cudaEvent_t e0,e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
  launch(out,cyc,nblk,threads); CK(cudaDeviceSynchronize());
  cudaEventRecord(e0); launch(out,cyc,nblk,threads); cudaEventRecord(e1); CK(cudaDeviceSynchronize());
  float ms; cudaEventElapsedTime(&ms,e0,e1);
  long long h[1024]; CK(cudaMemcpy(h,cyc,sizeof(long long)*nblk,cudaMemcpyDeviceToHost));
  double mx=0,avg=0; for(int i=0;i<nblk;i++){ if(h[i]>mx)mx=h[i]; avg+=h[i]; } avg/=nblk;
  double per_sm = (double)threads*ITERS*per_thread_per_iter;  // thread-level results per block(=SM)
  printf("%-28s blocks=%d thr=%d  cycles avg=%.0f max=%.0f  => %.2f %s/clk/SM ; time %.3f ms => eff clock %.0f MHz\n",
    name, nblk, threads, avg, mx, per_sm*unit_scale/avg, unit, ms, mx/ms/1e3);
  cudaFree(out); cudaFree(cyc);
  return 0;
}

int main(){
  cudaDeviceProp p; CK(cudaGetDeviceProperties(&p,0));
  printf("device %s cc %d.%d SMs %d clock %d kHz\n", p.name,p.major,p.minor,p.multiProcessorCount,p.clockRate);
  int n = p.multiProcessorCount;
  for (int threads : {256, 512, 1024}) {
    run("popc",        [](uint32_t*o,long long*c,int b,int t){k_pipe<0><<<b,t>>>(o,c,12345u);}, n, threads, 8, 1, "thread-instr");
    run("lop3",        [](uint32_t*o,long long*c,int b,int t){k_pipe<1><<<b,t>>>(o,c,12345u);}, n, threads, 8, 1, "thread-instr");
    run("iadd",        [](uint32_t*o,long long*c,int b,int t){k_pipe<2><<<b,t>>>(o,c,12345u);}, n, threads, 8, 1, "thread-instr");
    run("ffma",        [](uint32_t*o,long long*c,int b,int t){k_pipe<4><<<b,t>>>(o,c,12345u);}, n, threads, 8, 1, "thread-instr");
    run("xor+popc+add (words)", [](uint32_t*o,long long*c,int b,int t){k_pipe<3><<<b,t>>>(o,c,12345u);}, n, threads, 8, 1, "popc-words");
    run("popc+2lop3 (popc)", [](uint32_t*o,long long*c,int b,int t){k_pipe<5><<<b,t>>>(o,c,12345u);}, n, threads, 8, 1, "popc");
    run("popc+4lop3 (popc)", [](uint32_t*o,long long*c,int b,int t){k_pipe<6><<<b,t>>>(o,c,12345u);}, n, threads, 8, 1, "popc");
    run("mma b1 xor.popc", [](uint32_t*o,long long*c,int b,int t){k_bmma<0><<<b,t>>>(o,c,12345u);}, n, threads, 4.0/32, 16*8*256, "bit-MAC");
    run("mma b1 and.popc", [](uint32_t*o,long long*c,int b,int t){k_bmma<1><<<b,t>>>(o,c,12345u);}, n, threads, 4.0/32, 16*8*256, "bit-MAC");
    run("mma s8 m16n8k32", [](uint32_t*o,long long*c,int b,int t){k_imma<<<b,t>>>(o,c,12345u);}, n, threads, 4.0/32, 16*8*32, "MAC");
  }
  return 0;
}
