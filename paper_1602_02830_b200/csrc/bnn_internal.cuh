// Declarations shared between the library's translation units (not part of the public ABI).
#pragma once
#include "bnn_common.cuh"
#include "bnn_tile.cuh"

enum { BNN_VARIANT_AUTO = 0, BNN_VARIANT_PLAIN = 1, BNN_VARIANT_CSA = 2 };
static inline int ctx_variant(const bnn_ctx *ctx) { return ctx->variant; }

int bnn_launch_tile_packed(bnn_ctx *ctx, const bnn_tile::Args &a);
int bnn_launch_tile_conv(bnn_ctx *ctx, const bnn_tile::Args &a);
int bnn_launch_tile_planes(bnn_ctx *ctx, const bnn_tile::Args &a);
int bnn_output_scores(bnn_ctx *ctx, const uint32_t *Ap, int64_t lda_w, const uint32_t *Wp, int64_t ldw_w,
                      const float *gamma, const float *beta, const float *mean, const float *var, double eps,
                      float *scores, int64_t lds, int64_t M, int64_t N, int64_t K);

// ---- tensor-core int8 engine (bnn_umma.cu)
enum { BNN_ENGINE_AUTO = 0, BNN_ENGINE_POPC = 1, BNN_ENGINE_TENSOR = 2 };
size_t bnn_umma_operand_bytes(int64_t rows, int64_t K);   // bytes of an expanded (one byte per value) operand
int64_t bnn_umma_operand_ld(int64_t K);                   // its row pitch in bytes (multiple of 128)
int bnn_umma_expand(bnn_ctx *ctx, const uint32_t *src, int64_t ld_w, int64_t rows, int64_t K, int8_t *dst);
int bnn_umma_gemm(bnn_ctx *ctx, const void *A8, int64_t lda8, bool a_unsigned, const int8_t *B8, int64_t ldb8, int64_t M,
                  int64_t N, int64_t K, int32_t *C, int64_t ldc, const int32_t *thr, const uint32_t *flip, uint32_t *out,
                  int64_t ldo, int8_t *out8, int64_t ldo8, int pool = 0, int64_t H = 0, int64_t W = 0, int out_f4 = 0,
                  int b_static = 0);   // b_static: B8 is not written by the kernel launched just before (it may be read early)
// 4-bit (e2m1) operands: +-1 exactly, twice the MMA rate of the byte format (plain products only)
int64_t bnn_umma_operand_ld_f4(int64_t K);
size_t bnn_umma_operand_bytes_f4(int64_t rows, int64_t K);
int bnn_umma_expand_f4(bnn_ctx *ctx, const uint32_t *src, int64_t ld_w, int64_t rows, int64_t K, uint8_t *dst);
int bnn_umma_gemm_f4(bnn_ctx *ctx, const uint8_t *A4, int64_t lda4, const uint8_t *B4, int64_t ldb4, int64_t M, int64_t N,
                     int64_t K, int32_t *C, int64_t ldc, const int32_t *thr, const uint32_t *flip, uint32_t *out, int64_t ldo,
                     uint8_t *out4, int64_t ldo4, int b_static = 0);
int bnn_umma_im2col_u8(bnn_ctx *ctx, const uint8_t *act, int64_t B, int64_t H, int64_t W, int64_t C_in, uint8_t *dst);
// First convolution on the tensor engine: worth it from this many pixels / filters on.
static inline bool bnn_umma_first_conv_ok(int64_t pixels, int64_t C_out) { return pixels >= 16384 && C_out >= 64; }
// Shapes for which the tensor engine is worth its expansion pass.
static inline bool bnn_umma_shape_ok(int64_t M, int64_t N, int64_t K) {
    return M >= 256 && N >= 128 && K >= 128 && (double)M * (double)N * (double)K >= 1.0e9;
}
bool bnn_umma_conv_tiling(int64_t H, int64_t W, int pool, int *TH, int *TB);
int bnn_umma_conv(bnn_ctx *ctx, const int8_t *act8, const int8_t *W8, int64_t B, int64_t H, int64_t W, int64_t C_in,
                  int64_t C_out, int pool, const int32_t *thr, const uint32_t *flip, uint32_t *out_bits, int32_t *out_sums,
                  int8_t *out8 = nullptr, int64_t ldo8 = 0, int out_f4 = 0,   // out_f4: out8 receives e2m1 nibbles (ldo8 bytes per pixel)
                  int b_static = 0);                                          // b_static: W8 is not written by the kernel launched just before
bool bnn_umma_conv_f4_takes(const bnn_ctx *ctx, int64_t H, int64_t W, int pool, int64_t C_in);
int bnn_umma_conv_f4(bnn_ctx *ctx, const uint8_t *act4, const uint8_t *W4, int64_t B, int64_t H, int64_t W, int64_t C_in,
                     int64_t C_out, int pool, const int32_t *thr, const uint32_t *flip, uint32_t *out_bits, uint8_t *out4,
                     int64_t ldo4, int32_t *out_sums = nullptr, int b_static = 0);

// ---- bit-plane split as a pre-pass for the CUDA-core first layer (bnn_gemm.cu)
size_t bnn_planes_scratch_bytes(int64_t M, int64_t K);
int bnn_first_layer_planes_pre(bnn_ctx *ctx, const uint8_t *X, int64_t ldx, const uint32_t *Wp, int64_t ldw_w, const int32_t *thr,
                               const uint32_t *flip, uint32_t *out_bits, int64_t ldo_w, int32_t *out_sums, int64_t lds, int64_t M,
                               int64_t N, int64_t K, void *scratch);

// ---- filter repetitions (bnn_conv_fr.cu): only the distinct 2-D filters of every input channel are applied
size_t bnn_fr_workspace_bytes(int64_t C_in, int64_t C_out);
int bnn_fr_conv(bnn_ctx *ctx, const uint32_t *act, int64_t B, int64_t H, int64_t W, int64_t C_in, const uint32_t *Wp, int64_t C_out,
                int pool, const int32_t *thr, const uint32_t *flip, uint32_t *out_bits, int32_t *out_sums);
