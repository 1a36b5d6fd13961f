/*
 * bnn_b200 -- run-time path of Binarized Neural Networks on one NVIDIA B200 (sm_100a).
 *
 * C ABI.  Plain pointers and sizes only.
 *
 * Conventions (hold for every call unless a call says otherwise)
 *  - Every function returns an int status: BNN_OK (0) or a negative BNN_ERR_* code.  Nothing
 *    throws, aborts or exits.  Argument errors are reported before anything is launched.
 *  - Data pointers are DEVICE pointers owned by the caller.  The library never frees, keeps or
 *    reallocates them; they must stay valid until the work enqueued by the call has finished.
 *    Pointers marked "host" are host pointers.
 *  - Work is enqueued on the CUDA stream bound to the context and is asynchronous with respect
 *    to the host.  A context may be used by one host thread at a time.
 *  - A +-1 value is stored as one bit: bit 1 <-> +1, bit 0 <-> -1 (bit = (x >= 0), Eq. 1).
 *    Element k of a row sits in 32-bit word k/32 at bit k%32 (least significant bit first);
 *    a 64-bit word j is words 2j and 2j+1, so both word widths are the same bytes in memory
 *    (Section 4: 32 binary variables concatenated per register).
 *  - "Packed matrix R x K": R rows, each ceil(K/32) words, leading dimension ld_w words with
 *    ld_w >= ceil(K/32) and ld_w % 4 == 0, base address 16-byte aligned (BNN_ERR_ALIGNMENT
 *    otherwise).  Bits at positions >= K of the last word and words beyond ceil(K/32) are
 *    padding: producers write them as 0, consumers ignore them whatever they hold.
 *  - Sizes are int64_t.  A dimension of 0 is legal: the call is a no-op (M or N == 0) or yields
 *    the empty sum 0 (K == 0).
 */
#ifndef BNN_B200_H
#define BNN_B200_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define BNN_API __attribute__((visibility("default")))
#else
#define BNN_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

enum {
    BNN_OK = 0,
    BNN_ERR_INVALID_ARG = -1,   /* NULL pointer, negative size, unknown enum value, ld too small   */
    BNN_ERR_ALIGNMENT = -2,     /* base pointer or leading dimension breaks the alignment rule     */
    BNN_ERR_WORKSPACE = -3,     /* workspace missing or too small                                   */
    BNN_ERR_CUDA = -4,          /* a CUDA runtime call failed; see bnn_last_cuda_error()            */
    BNN_ERR_DEVICE_STATUS = -5, /* a kernel reported an internal error through its status word      */
    BNN_ERR_TOO_LARGE = -6      /* bnn_mlp_forward_noalloc: the problem does not fit the built-in scratch */
};

enum { BNN_F32 = 0, BNN_F16 = 1, BNN_I8 = 2 }; /* element type of bnn_pack_signs' source */

typedef struct bnn_ctx bnn_ctx;

/* Context = (device, stream, optional caller-owned workspace).  `cuda_stream` is a cudaStream_t
 * (NULL = the legacy default stream).  The context owns no device memory. */
BNN_API int bnn_create(bnn_ctx **out, int device, void *cuda_stream);
BNN_API int bnn_destroy(bnn_ctx *ctx);
BNN_API const char *bnn_status_string(int status);
/* cudaError_t of the most recent failing CUDA call made through this context (0 if none). */
BNN_API int bnn_last_cuda_error(const bnn_ctx *ctx);
/* Lend `bytes` of device memory (256-byte aligned) to the context for calls that need scratch
 * (bnn_mlp_forward, bnn_mlp_forward_host).  Pass NULL, 0 to take it back. */
BNN_API int bnn_set_workspace(bnn_ctx *ctx, void *dptr, size_t bytes);
/* Inner loop of the tiled kernels (results are identical): 0 = library default, 1 = one POPC per
 * word (Eq. 8 as written), 2 = carry-save: a LOP3 full adder merges two XOR words before the POPC. */
BNN_API int bnn_set_popc_variant(bnn_ctx *ctx, int variant);
/* Accumulator rows per thread of the tiled CUDA-core kernel: 16 (one CTA of 8 warps per SM) or 8 (two CTAs per
 * SM, more warps per scheduler; the default, faster on B200).  A tuning knob; results are identical. */
BNN_API int bnn_set_tile_rows(bnn_ctx *ctx, int rows);

/* Which kernels evaluate the large products (results are the same integers either way):
 *   0 = automatic: the tensor-core engine for large shapes when the context's workspace is big enough
 *       (bnn_gemm_workspace_bytes / bnn_mlp_workspace_bytes), otherwise the CUDA-core kernels;
 *   1 = CUDA-core XOR-popcount kernels only (Eq. 8 as the paper computes it);
 *   2 = tensor-core engine wherever the shape qualifies; BNN_ERR_WORKSPACE if the workspace is too small.
 * The tensor-core engine expands the packed operands in the workspace to the format bnn_set_operand_bits selects
 * (4-bit e2m1 nibbles by default, signed bytes for layers with 8-bit inputs) and multiplies them exactly with
 * tcgen05 tensor-core instructions (Section 4: on +-1 inputs the binary kernel and an ordinary matrix product
 * return identical outputs).  Engine 1 is the XOR-popcount form the popc roofline applies to. */
BNN_API int bnn_set_engine(bnn_ctx *ctx, int engine);
/* Tensor-core engine only: plain products can run on pairs of SMs (thread-block clusters of two, tcgen05
 * cta_group::2) that share the B operand.  0 (default) = for outputs of 6 million elements and more, where it measured
 * faster; 1 = never; 2 = wherever the kernel allows (M >= 512; also the 4-bit convolutions).  Results are identical. */
BNN_API int bnn_set_pair_mode(bnn_ctx *ctx, int mode);
/* Tensor-core engine only: how +-1 x +-1 products are fed to the tensor cores.  4 (default) = each value as a 4-bit
 * floating-point nibble (e2m1: +-1.0 is exact, block scales fixed at 1, float32 accumulators that hold these integer sums
 * exactly for K <= 2^24): half the operand bytes and twice the instruction rate of 8 = one signed byte per value with
 * int32 accumulators.  Layers with 8-bit inputs always use bytes, and so do convolutions whose C_in is not a multiple
 * of 256 (a K step of the 4-bit kernel is 256 channels of one tap).  Results are identical. */
BNN_API int bnn_set_operand_bits(bnn_ctx *ctx, int bits);
/* Workspace bytes bnn_xnor_gemm / bnn_binary_dense need to run M x N x K on the tensor-core engine
 * (0 if the shape does not qualify for it). */
BNN_API size_t bnn_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K);
/* The same for bnn_binary_conv2d (0 if the tensor-core engine does not apply: a binary input needs
 * C_in % 128 == 0 and a width that divides 128; 9 * C_in <= 32 means the 8-bit first layer). */
BNN_API size_t bnn_conv_workspace_bytes(int64_t B, int64_t H, int64_t W, int64_t C_in, int64_t C_out, int pool);
/* Packed signs -> one signed byte per value (+1 -> 0x01, -1 -> 0xff), the operand format of the tensor-core engine.
 *   src packed rows x K (ld_w words); dst rows x bnn_expanded_ld(K) bytes, bytes at positions >= K written as 0;
 *   dst must be 16-byte aligned and hold bnn_expanded_bytes(rows, K).  Weights can be expanded once and handed to
 *   bnn_mlp_forward through bnn_layer_desc.W8. */
BNN_API int64_t bnn_expanded_ld(int64_t K);
BNN_API size_t bnn_expanded_bytes(int64_t rows, int64_t K);
BNN_API int bnn_expand_signs(bnn_ctx *ctx, const uint32_t *src, int64_t ld_w, int64_t rows, int64_t K, int8_t *dst);
/* The same as 4-bit floating-point nibbles (e2m1: +1 -> 0x2, -1 -> 0xa, two values per byte, value k in byte k/2 with
 * even k in the low nibble; nibbles at positions >= K are 0).  Row pitch bnn_expanded_ld_f4(K) bytes. */
BNN_API int64_t bnn_expanded_ld_f4(int64_t K);
BNN_API size_t bnn_expanded_bytes_f4(int64_t rows, int64_t K);
BNN_API int bnn_expand_signs_f4(bnn_ctx *ctx, const uint32_t *src, int64_t ld_w, int64_t rows, int64_t K, uint8_t *dst);
/* Hidden layer (Algorithm 4: product, BatchNorm folded to thr / flip, Sign) on operands that are already in an
 * expanded format, i.e. the tensor-core kernel of bnn_binary_dense without its two expansion passes: for callers that
 * keep weights and activations expanded, as bnn_mlp_forward does between its layers.
 *   operand_bits 8: A_exp M x K and W_exp N x K as written by bnn_expand_signs (pitches in bytes, multiples of 16);
 *   operand_bits 4: as written by bnn_expand_signs_f4 (K <= 2^24).
 *   out_bits (optional): packed M x N signs, pitch ldo_w words, like bnn_binary_dense.
 *   out_exp  (optional): the same signs in the operand format of the next layer (same operand_bits), pitch
 *                        ldo_exp bytes >= bnn_expanded_ld(N) or bnn_expanded_ld_f4(N); at least one output is required.
 *                        Values N .. roundup(N, 32) - 1 of a row are written as 0 (all that a following layer with
 *                        K = N reads); the rest of the pitch is left untouched.
 * Runs on the context's stream; BNN_ERR_ALIGNMENT for pointers or pitches that are not multiples of 16 bytes. */
BNN_API int bnn_binary_dense_expanded(bnn_ctx *ctx, const void *A_exp, int64_t lda_bytes, const void *W_exp, int64_t ldw_bytes,
                                      int operand_bits, const int32_t *thr, const uint32_t *flip, uint32_t *out_bits,
                                      int64_t ldo_w, void *out_exp, int64_t ldo_exp, int64_t M, int64_t N, int64_t K);
/* Tensor-core engine only: how a 3x3 convolution brings its input into shared memory.  0 (default) = halo tiles: per
 * tile and horizontal tap one slab of TH + 2 image rows, read at three row offsets for the three vertical taps (a
 * third of the input traffic; the tile's weights stay resident where they fit); 1 = one 128-pixel operand box per tap.
 * Geometries the halo form does not cover (tile rows that are not whole 1024-byte groups) use form 1 either way.
 * Results are identical. */
BNN_API int bnn_set_conv_form(bnn_ctx *ctx, int form);
/* Tensor-core engine only: every wait of its kernels on a barrier (operands arrived, stage free, accumulator ready) is
 * bounded.  A wait that lasts longer than `ns` nanoseconds of wall clock (default 2 s; 1 .. 60 s) gives up: the kernel
 * records a code, skips the rest of its work, frees its tensor memory and ends normally, and the other waiters of the
 * same CTA (and of its partner in a CTA pair) stop at their next look, so one failure costs about one limit.
 * bnn_device_status then reports BNN_ERR_DEVICE_STATUS and the context stays usable. */
BNN_API int bnn_set_wait_limit_ns(bnn_ctx *ctx, uint64_t ns);
/* Test hook for the failure path above (host-side injection, nothing faults): while on = 1 the tensor-core kernels
 * launched through this context run in their single-SM form with a producer that requests no operands, so their
 * consumers' waits run into the limit.  Outputs of such calls are undefined.  on = 0 restores normal operation. */
BNN_API int bnn_debug_drop_loads(bnn_ctx *ctx, int on);
/* Test hook, host only (no context, no GPU): where stage number `stage` (0, 1, 2, ... in the order a CTA's producer fills
 * them) of a tensor-engine operand ring of `slots` slots lives.  The kernels guard every slot with TWO barrier pairs, used
 * alternately, so that each barrier has a single consuming thread when two threads issue alternate stages: stage G uses
 * slot G mod slots, barrier pair G mod (2 slots), and waits for phase parity (G div (2 slots)) mod 2.
 * Outputs: the stage's slot, barrier pair and parity; whether an earlier stage used the slot (reuses) and, if so, the
 * barrier pair and parity of that stage (stage - slots), which the producer waits for before refilling; and the barrier
 * pair and parity after advancing by `step` stages (1 <= step <= 2 slots), as a thread that takes every step-th stage does.
 * BNN_ERR_INVALID_ARG for slots = 0, step out of range or a null pointer. */
BNN_API int bnn_debug_ring_position(uint32_t stage, uint32_t slots, uint32_t step, uint32_t *slot, uint32_t *barrier,
                                    uint32_t *parity, int32_t *reuses, uint32_t *prev_barrier, uint32_t *prev_parity,
                                    uint32_t *next_barrier, uint32_t *next_parity);
/* Synchronises the context's stream and returns BNN_ERR_DEVICE_STATUS if a kernel gave up on one of its
 * bounded waits since the last call (its outputs are then undefined), BNN_OK otherwise. */
BNN_API int bnn_device_status(bnn_ctx *ctx);

/* ---------------------------------------------------------------------------------------------
 * Sign-pack (Eq. 1 followed by the 32-per-word concatenation of Section 4).
 *   src        rows x cols elements of `dtype`, row-major, leading dimension src_ld elements.
 *   pack_along 0: pack along cols -> dst is a packed matrix rows x cols   (e.g. A, activations)
 *              1: pack along rows -> dst is a packed matrix cols x rows   (a K x N weight matrix
 *                 becomes the N x K packed operand the GEMM calls expect)
 *   word_bits  32 or 64 (same bytes; 64 additionally needs dst_ld_w even).
 *   dst        packed matrix, leading dimension dst_ld_w words.  All padding is written as 0.
 * bit = (x >= 0); both zeros give 1.  NaN is not a legal input.
 */
BNN_API int bnn_pack_signs(bnn_ctx *ctx, const void *src, int dtype, int64_t rows, int64_t cols, int64_t src_ld,
                   int pack_along, int word_bits, uint32_t *dst, int64_t dst_ld_w);

/* ---------------------------------------------------------------------------------------------
 * Binary matrix product (Section 4, Eq. 8).  C[m][n] = sum_k A[m][k] * B[k][n] over +-1 values
 *   = K - 2 * popcount(Ap[m] XOR Bp[n]).
 *   Ap packed M x K (lda_w), Bp packed N x K (ldb_w: B is given transposed, K along words),
 *   C  M x N int32 row-major, leading dimension ldc >= N elements.
 */
BNN_API int bnn_xnor_gemm(bnn_ctx *ctx, const uint32_t *Ap, int64_t lda_w, const uint32_t *Bp, int64_t ldb_w,
                  int32_t *C, int64_t ldc, int64_t M, int64_t N, int64_t K);

/* ---------------------------------------------------------------------------------------------
 * Hidden layer (Algorithm 4, step 2): binary product fused with the BatchNorm-folded integer
 * threshold, Sign (Eq. 1) and repacking.  out_bit[m][n] = (dot[m][n] >= thr[n]) XOR flip_bit[n].
 *   Ap packed M x K, Wp packed N x K, thr N int32 (any value), flip packed 1 x N or NULL (all 0),
 *   out packed M x N (ldo_w words; padding written as 0).  No int32 product is written.
 */
BNN_API int bnn_binary_dense(bnn_ctx *ctx, const uint32_t *Ap, int64_t lda_w, const uint32_t *Wp, int64_t ldw_w,
                     const int32_t *thr, const uint32_t *flip, uint32_t *out, int64_t ldo_w, int64_t M,
                     int64_t N, int64_t K);

/* ---------------------------------------------------------------------------------------------
 * First layer on 8-bit inputs (Section 1.6, Eq. 6-7; Algorithm 4, step 1):
 *   s[m][n] = sum_i X[m][i] * w[i][n] = sum_{p=1..8} 2^(p-1) * (x^p[m] . w[:,n]),  x^p in {0,1}.
 *   X  M x K uint8 row-major (ldx elements), Wp packed N x K.  The tensor-core engine needs X 16-byte aligned and
 *      ldx a multiple of 16 (otherwise the CUDA-core kernels run); rows that start on 32-byte boundaries (ldx a
 *      multiple of 32, e.g. 800 for K = 784) are fetched in whole sectors and make the layer about 15 % faster.
 *   out_sums (or NULL): M x N int32, leading dimension lds.
 *   out_bits (or NULL): packed M x N, bit = (s >= thr[n]) XOR flip_bit[n]; thr is required then.
 * At least one output must be given.
 */
BNN_API int bnn_first_layer_bitplanes(bnn_ctx *ctx, const uint8_t *X, int64_t ldx, const uint32_t *Wp, int64_t ldw_w,
                              const int32_t *thr, const uint32_t *flip, uint32_t *out_bits, int64_t ldo_w,
                              int32_t *out_sums, int64_t lds, int64_t M, int64_t N, int64_t K);

/* ---------------------------------------------------------------------------------------------
 * Binary 3x3 convolution, stride 1, one pixel of padding, as an implicit GEMM (Section 3.3).
 * A tap that falls outside the image contributes 0.  Optional 2x2 / stride-2 max-pooling of the
 * integer sums, then bit = (sum >= thr[n]) XOR flip_bit[n].
 *   act     binary input, NHWC, channels packed: [B][H][W][C_in/32] words (C_in % 32 == 0), or
 *   act_u8  8-bit input for a first layer, NHWC [B][H][W][C_in] bytes, 9*C_in <= 32 (bit-planes);
 *           exactly one of act / act_u8 is non-NULL.
 *   Wp      [C_out][3][3][C_in/32] words for a binary input; for act_u8 one word per filter with
 *           bit (tap*C_in + c), tap = 3*(dy+1) + (dx+1).
 *   pool    0 or 1 (H and W must be even when 1).  Output height/width are H, W or H/2, W/2.
 *   out_bits (or NULL) [B][Ho][Wo][ceil(C_out/32)] words; out_sums (or NULL) [B][Ho][Wo][C_out] int32
 *           (pooled sums when pool == 1).  thr is required when out_bits is given.
 */
BNN_API int bnn_binary_conv2d(bnn_ctx *ctx, const uint32_t *act, const uint8_t *act_u8, int64_t B, int64_t H,
                      int64_t W, int64_t C_in, const uint32_t *Wp, int64_t C_out, int pool,
                      const int32_t *thr, const uint32_t *flip, uint32_t *out_bits, int32_t *out_sums);

/* ---------------------------------------------------------------------------------------------
 * Exploiting filter repetitions (Section 3.3).  A binary 3x3 filter over C_in channels consists of C_in two-dimensional
 * 3x3 filters, of which only 2^9 exist -- 2^8 classes when a filter and its negation count as one.  With the switch on,
 * bnn_binary_conv2d on a binary input classifies the layer's C_out x C_in 2-D filters, applies per input channel only the
 * DISTINCT ones to the map (one XNOR-popcount on a 9-bit neighbourhood per distinct filter and pixel) and forms every
 * filter's result as a signed sum of those responses.  Results are the same integers and bits as without the switch.
 * It runs on the CUDA cores and needs a workspace of bnn_filter_repetition_workspace_bytes(C_in, C_out) for the class
 * tables (BNN_ERR_WORKSPACE otherwise).  It shows the mechanism; on this GPU the full product on the tensor cores is faster.
 * bnn_filter_repetition_count classifies the filters Wp ([C_out][3][3][C_in / 32] words) and returns, in *distinct (host),
 * the number of distinct 2-D filters summed over the input channels (at most min(256, C_out) per channel, against
 * C_out * C_in filter applications without the exploit); it uses the same workspace and synchronises the stream. */
BNN_API int bnn_set_conv_filter_repetition(bnn_ctx *ctx, int on);
BNN_API size_t bnn_filter_repetition_workspace_bytes(int64_t C_in, int64_t C_out);
BNN_API int bnn_filter_repetition_count(bnn_ctx *ctx, const uint32_t *Wp, int64_t C_in, int64_t C_out, int64_t *distinct);

/* ---------------------------------------------------------------------------------------------
 * Whole ConvNet forward: a stack of 3x3 / pad-1 layers, each  conv -> optional 2x2 max-pool -> threshold -> Sign
 * (Algorithm 4 with convolutions in place of the dense products, Section 3.3).  Layer 0 takes the 8-bit image
 * (9 * C_in <= 32, bit-plane layer of Section 1.6); every other layer takes the previous layer's binary map.
 * The activations stay on the device between layers (packed, plus one byte per value for the tensor-core engine).
 */
typedef struct {
    const uint32_t *Wp;   /* as for bnn_binary_conv2d (device) */
    int64_t C_in, C_out;
    int32_t pool;         /* 0 or 1 */
    const int32_t *thr;   /* C_out thresholds (device) */
    const uint32_t *flip; /* packed 1 x C_out or NULL (device) */
    const int8_t *W8;     /* optional (device, may be NULL): bnn_expand_signs(Wp viewed as C_out rows of 9*C_in bits) */
    const uint8_t *W4;    /* optional (device, may be NULL): bnn_expand_signs_f4 of the same rows; read instead of W8 by
                             layers whose C_in is a multiple of 256 (they run on 4-bit operands unless
                             bnn_set_operand_bits(ctx, 8) was called) */
} bnn_conv_layer_desc;

typedef struct {
    int32_t n_layers;
    const bnn_conv_layer_desc *layers; /* host array */
} bnn_convnet_desc;

BNN_API size_t bnn_convnet_workspace_bytes(const bnn_convnet_desc *net, int64_t B, int64_t H, int64_t W);
/* X: [B][H][W][C_in of layer 0] bytes (device).  out_bits: the last layer's packed map [B][Ho][Wo][ceil(C_out/32)].
 * layer_out: NULL, or a host array of n_layers device pointers (entries may be NULL) that receive every layer's packed
 * map.  Needs a workspace of bnn_convnet_workspace_bytes (BNN_ERR_WORKSPACE otherwise). */
BNN_API int bnn_convnet_forward(bnn_ctx *ctx, const bnn_convnet_desc *net, const uint8_t *X, int64_t B, int64_t H, int64_t W,
                                uint32_t *out_bits, uint32_t *const *layer_out);

/* ---------------------------------------------------------------------------------------------
 * Whole MLP forward (Algorithm 4): first layer on 8-bit inputs, hidden binary layers, real-valued
 * output layer  score = gamma * ((dot - mean) / sqrt(var + eps)) + beta  (evaluated in double as
 * dot * a + b with a = gamma / sqrt(var + eps), b = beta - mean * a, rounded once to float32).
 */
typedef struct {
    const uint32_t *Wp;  /* packed N x K weights (device) */
    int64_t ldw_w;
    int64_t K, N;
    const int32_t *thr;  /* hidden layers: N thresholds (device) */
    const uint32_t *flip; /* hidden layers: packed 1 x N or NULL (device) */
    const float *gamma, *beta, *mean, *var; /* output layer only: N floats each (device) */
    double eps;                             /* output layer only */
    const int8_t *W8; /* optional (device, may be NULL): the same weights as written by bnn_expand_signs, used by the
                         tensor-core engine; when NULL that engine expands Wp into the workspace on every call */
    const uint8_t *W4; /* optional (device, may be NULL): the same weights as written by bnn_expand_signs_f4; what the
                          tensor-core engine reads for layers 2.. when the operand width is 4 bits (the default) */
} bnn_layer_desc;

typedef struct {
    int32_t n_layers;             /* >= 2: first layer, hidden layers..., output layer */
    const bnn_layer_desc *layers; /* host array of n_layers entries */
} bnn_mlp_desc;

/* Scratch bytes bnn_mlp_forward (host_io = 0) or bnn_mlp_forward_host (host_io = 1) need for `batch`. */
BNN_API size_t bnn_mlp_workspace_bytes(const bnn_mlp_desc *m, int64_t batch, int host_io);
/* X batch x K0 uint8 (device, ldx; see bnn_first_layer_bitplanes for what ldx means to the tensor-core engine),
 * scores batch x N_last float32 (device, lds).
 * If `hidden_out` is not NULL it is a host array of n_layers-1 device pointers (entries may be NULL);
 * hidden layer k's packed activations (batch x N_k, leading dimension ceil(N_k/128)*4 words)
 * are also copied there.  Needs a workspace (BNN_ERR_WORKSPACE otherwise). */
BNN_API int bnn_mlp_forward(bnn_ctx *ctx, const bnn_mlp_desc *m, const uint8_t *X, int64_t ldx, int64_t batch,
                    float *scores, int64_t lds, uint32_t *const *hidden_out);
/* Same with HOST input and output: X_host is copied to the device and the scores are copied back (pinned host
 * memory makes the copies asynchronous).  For large batches the input travels in row chunks on an internal stream
 * so that later chunks are copied while earlier ones are already being computed; all of it is ordered after the work
 * already queued on the context's stream and completes before anything queued on it afterwards, so the caller just
 * synchronises the context's stream. */
BNN_API int bnn_mlp_forward_host(bnn_ctx *ctx, const bnn_mlp_desc *m, const uint8_t *X_host, int64_t ldx,
                         int64_t batch, float *scores_host, int64_t lds);

/* ---------------------------------------------------------------------------------------------
 * Measurement helper (Section 4 counts the XNOR-popcount step as "1 + 4 + 1" cycles on the GPUs of 2016): the issue rates
 * of this GPU's integer pipes, in thread-level results per clock and SM, timed in register-only loops on every SM:
 * POPC alone, LOP3 alone, and the xor / popc / add sequence of Eq. 8 (counted per popcount word).  The popcount roofline
 * of a benchmark is  SMs x popc rate x 32 bit-MACs x 2 x SM clock.
 *   scratch: device memory, at least sm_count * 4104 bytes, 8-byte aligned (BNN_ERR_WORKSPACE / BNN_ERR_ALIGNMENT).
 * Runs on the context's stream and synchronises it; the three results are host doubles. */
BNN_API int bnn_measure_pipe_rates(bnn_ctx *ctx, void *scratch, size_t scratch_bytes, double *popc_per_clk_per_sm,
                                   double *lop3_per_clk_per_sm, double *xor_popc_add_per_clk_per_sm);
/* Name and tile shape of the tensor-core kernel this context launched last ("" if none yet): lets a benchmark label its
 * numbers with what actually ran.  The string is owned by the context and valid until its next call. */
BNN_API const char *bnn_last_tensor_kernel(const bnn_ctx *ctx);
/* The SM clock the tensor-core kernel launched last on this device really ran at, and how long its first CTA lived:
 * the kernel's CTA 0 reads the SM cycle counter and the nanosecond timer when it starts and when it ends.  (This part
 * holds tensor-heavy kernels well below the maximum SM clock that nvidia-smi samples around them.)  Synchronises the
 * context's stream.  sm_mhz, microseconds: host pointers, written.  0.0 MHz if no such kernel has run. */
BNN_API int bnn_last_tensor_kernel_clock(bnn_ctx *ctx, double *sm_mhz, double *microseconds);

/* ---------------------------------------------------------------------------------------------
 * Context only (Section 4, Fig. 3): the paper's comparison point, a deliberately unoptimized matrix product of the
 * +-1 values held as float32 (one thread per output).  A is M x K, B is K x N, C is M x N, all row-major device
 * float32.  Not used by any other call. */
BNN_API int bnn_baseline_gemm_f32(bnn_ctx *ctx, const float *A, const float *B, float *C, int64_t M, int64_t N,
                                  int64_t K);

/* ---------------------------------------------------------------------------------------------
 * bnn_mlp_forward for callers that cannot allocate device memory.  (The paper has no counterpart: this
 * is a deployment convenience of the library, not a step of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a serving loop whose device memory was
 * sized and handed out at start-up and whose policy forbids further allocation (an allocation can
 * synchronise the device, fail under memory pressure, or fragment a pool someone else owns), a plug-in
 * that is handed pointers but owns no allocator, or a process that simply has no memory budget left for a
 * workspace.  Such a caller still passes its input and output buffers; only the scratch between the layers
 * is supplied by the library, from an array that is part of the library image.
 *
 * Same arguments and results as bnn_mlp_forward (device X and scores; no hidden_out), no workspace needed
 * and none used: a workspace that was lent to the context for other calls is neither read nor written.
 * Limits and rules:
 *  - batch * ceil(widest hidden layer / 128) * 16 bytes must not exceed bnn_mlp_noalloc_max_bytes()
 *    (512 KiB: e.g. batch 1024 at 4096 units); beyond that the call returns BNN_ERR_TOO_LARGE and does nothing.
 *    Every GPU that loads the library holds 1 MiB for this array until the process exits.
 *  - The first call on each device looks up the array's device address (one cudaGetSymbolAddress, no
 *    allocation); make that first call before starting any stream capture on that device.
 *  - The call itself never calls cudaMalloc, cudaFree or any allocating routine.
 *  - All calls on one device share the one array: calls whose GPU work can overlap (different streams,
 *    different contexts, different threads) race on it and must be serialised by the caller.  The array
 *    keeps whatever the last call left; no call depends on its previous contents.
 */
BNN_API size_t bnn_mlp_noalloc_max_bytes(void);
BNN_API int bnn_mlp_forward_noalloc(bnn_ctx *ctx, const bnn_mlp_desc *m, const uint8_t *X, int64_t ldx,
                                    int64_t batch, float *scores, int64_t lds);

/* ---------------------------------------------------------------------------------------------
 * Host helper (not on the timed path): fold run-time BatchNorm followed by Sign,
 *   Sign(gamma * ((x - mean) / sqrt(var + eps)) + beta)   evaluated in double for integer x,
 * into the integer rule (x >= thr[n]) XOR flip_bit[n] that is exact for every integer |x| <= x_max.
 * All pointers are HOST pointers; flip is packed 1 x n (ceil(n/32) words).
 */
BNN_API int bnn_fold_batchnorm(const float *gamma, const float *beta, const float *mean, const float *var, double eps,
                       int64_t n, int64_t x_max, int32_t *thr, uint32_t *flip);

#ifdef __cplusplus
}
#endif
#endif /* BNN_B200_H */
