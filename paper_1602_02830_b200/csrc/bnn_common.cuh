// Shared host-side plumbing of the bnn_b200 library: context, status codes, argument checks.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>
#include <stdio.h>
#include "bnn_b200.h"

struct bnn_ctx {
    int device;
    cudaStream_t stream;
    void *ws;
    size_t ws_bytes;
    int last_cuda_error;
    int sm_count;
    int variant;   // inner-loop choice of the tiled kernel (0 auto, 1 plain popc, 2 carry-save)
    int tile_rows; // accumulator rows per thread of the tiled popc kernel: 16 or 8
    int pair_mode; // tensor engine: 0 = CTA pairs (cta_group::2) for very large outputs, 1 = never, 2 = wherever the kernel allows
    cudaStream_t copy_stream;   // internal stream for the host copies of bnn_mlp_forward_host (created on first use)
    cudaEvent_t ev[8];          // [0] work already on `stream`; [1..4] chunk copies done; [5] chunk computed; [6] scores copied
    bool copy_ready;
    int operand_bits; // tensor engine, +-1 x +-1 products: 4 = e2m1 nibbles (default), 8 = signed bytes
    int engine;    // 0 auto, 1 CUDA-core XOR-popcount kernels only, 2 tensor-core int8 engine where it applies
    unsigned long long wait_limit_ns;   // tensor engine: how long one of its device-side waits may last before it gives up
    int filter_repetition;   // bnn_binary_conv2d on a binary input applies only the distinct 2-D filters per channel (Section 3.3)
    int conv_form;    // tensor engine, 3x3 convolutions: 0 = halo-tile kernel where the geometry allows, 1 = one operand box per tap
    char last_kernel[160];   // the tensor-core kernel launched last, for bnn_last_tensor_kernel
    int drop_loads;   // test hook: the tensor kernels' producer issues no loads, so that their waits run into the limit
};

#define BNN_CUDA_TRY(ctx, call)                              \
    do {                                                     \
        cudaError_t e__ = (call);                            \
        if (e__ != cudaSuccess) {                            \
            if (ctx) (ctx)->last_cuda_error = (int)e__;      \
            return BNN_ERR_CUDA;                             \
        }                                                    \
    } while (0)

// Programmatic dependent launch: the kernel may be set up on the GPU while its predecessor in the stream still runs.
// Kernels launched this way call bnn_pdl_wait() before their first access to global memory; it returns once the
// predecessor has completed and its writes are visible (immediately for an ordinary launch).  They release their own
// successor (bnn_pdl_launch_next) only after that wait, so by the time a kernel runs at all, everything older than its
// immediate predecessor is complete: the only data a kernel may touch before its wait is data that the immediately
// preceding kernel does not write (weights and parameters prepared earlier).
template <typename... KArgs, typename... Args>
static inline cudaError_t bnn_launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                               Args &&...args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#ifdef __CUDACC__
__device__ __forceinline__ void bnn_pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel of the stream be set up as soon as every CTA of this one has got here (it still waits in
// bnn_pdl_wait for this kernel to finish before it touches memory).
__device__ __forceinline__ void bnn_pdl_launch_next() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif

static inline int bnn_check_launch(bnn_ctx *ctx) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        ctx->last_cuda_error = (int)e;
        return BNN_ERR_CUDA;
    }
    return BNN_OK;
}

static inline int64_t bnn_words(int64_t k) { return (k + 31) / 32; }
static inline bool bnn_aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// A packed matrix R x K with leading dimension ld_w: checks of the ABI's layout rule.
static inline int bnn_check_packed(const void *p, int64_t ld_w, int64_t K, int64_t R) {
    if (R == 0) return BNN_OK;
    if (p == nullptr) return BNN_ERR_INVALID_ARG;
    if (ld_w < bnn_words(K) || ld_w < 0) return BNN_ERR_INVALID_ARG;
    if (!bnn_aligned16(p) || (ld_w % 4) != 0) return BNN_ERR_ALIGNMENT;
    return BNN_OK;
}

// Keeps `ctx`'s device current for the duration of a call and restores the caller's device after.
struct bnn_device_guard {
    int prev = -1;
    bool ok = true;
    explicit bnn_device_guard(bnn_ctx *ctx) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != ctx->device && cudaSetDevice(ctx->device) != cudaSuccess) ok = false;
    }
    ~bnn_device_guard() { if (prev >= 0) cudaSetDevice(prev); }
};
