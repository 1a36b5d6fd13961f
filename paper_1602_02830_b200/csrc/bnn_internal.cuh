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
