// Tensor-core engine for the large products: the +-1 (or 8-bit x +-1) product evaluated EXACTLY by the
// 5th-generation tensor cores, accumulators in tensor memory.
//
//   Section 4 states that the binary kernel and an ordinary matrix product return identical outputs on +-1
//   inputs.  On sm_100a the ordinary product has a far higher ceiling than the POPC pipe (8192 int8 or 16384
//   4-bit MACs against 512 bit-MACs per clock per SM), so for large shapes the packed operands are expanded
//   (a streaming pass) and multiplied on the tensor cores.  Results are the same integers.
//     bytes   (+1 = 0x01, -1 = 0xff; the 8-bit first layer's pixels as they are): tcgen05.mma kind::i8, int32
//             accumulators, 128 x 256 tiles (128 x 128 for narrow outputs);
//     nibbles (e2m1: +1 = 0x2, -1 = 0xa): tcgen05.mma kind::mxf4.block_scale with every block scale 2^0 (32 TMEM
//             columns filled once with the UE8M0 byte 0x7f), float32 accumulators (exact while K <= 2^24),
//             128 x 192 tiles (CTA pairs: 256 x 192 or 256 x 224), twice the MMA rate and half the operand bytes.
//
// Kernel k_umma_i8<BN> (persistent, one CTA per SM walking 128 x BN output tiles, column blocks fastest):
//   warp 0       TMA producer: cp.async.bulk.tensor loads of 128-byte-wide K slices (128B swizzle) of both
//                operands into a ring of 4-6 shared-memory stages, completion on mbarriers;
//   warp 1 and the last warp  MMA issuers: one lane each, alternate K steps of every tile (issuing a step costs one
//                thread more clocks than the tensor core needs to run it); four MMAs per step, tcgen05.commit
//                releases the stage; warp 1 also allocates the TMEM columns (two accumulator buffers);
//   warps 2 ..   epilogue, 8 warps on the 4-bit tiles (two per TMEM lane quadrant, each a contiguous half of the
//                columns, the next 32-column chunk in flight while the current one is processed), 16 on the byte
//                tiles (four per quadrant): tcgen05.ld of the accumulators (one output row per thread), then int32
//                stores, or the BatchNorm-folded threshold + Sign as one 32-bit word per 32 columns and/or the same
//                signs in the next layer's operand format.
// Kernel k_umma_i8_2sm<BN>: the same with a cluster of two CTAs on one 256 x BN tile (cta_group::2); BN = 256 or 128
// for bytes, 192 or 224 for nibbles (224: the widest tile whose two accumulator buffers and scale columns fit tensor
// memory; its K step brings 240 operand rows for 448 clocks of MMAs, which L2 can deliver, see bnn_umma_gemm_f4).
// Every wait is bounded: after the limit the kernel records an error code and runs to its end without
// touching the accumulators, so a failure surfaces as BNN_ERR_DEVICE_STATUS instead of a hang.
#include "bnn_internal.cuh"
#include <cuda.h>
#include <mutex>

namespace {

constexpr int BM = 128, BK = 128;               // BK in bytes = int8 elements
constexpr int BN_MAX = 256;                     // tile width: 256, or 128 for narrow outputs; 192 = the 4-bit engine
constexpr uint32_t SF_COL = 480;                // 4-bit engine: first of the 32 TMEM columns that hold the scale factors
// Tile widths of the 4-bit engine: 192, and 224 for the pair kernel (two accumulator buffers + 32 scale columns <= 512)
constexpr bool is_f4(int bn) { return bn == 192 || bn == 224; }
constexpr int N_ISSUE = 2;                      // MMA-issuing warps: warp 1 and the warps behind the epilogue warps
// Epilogue warps per tile width: EPW per TMEM lane quadrant.  With two, each takes a contiguous half of the columns and
// prefetches its next chunk; with four, chunks go round-robin and the other warps of the scheduler cover the load
// latency (one register buffer, so the kernel fits 608 threads).  Four measured faster where signs are the output of
// 256- and 128-wide tiles (first layer of the MLP, convolutions), two where int32 sums are stored (the 192-wide GEMM).
template <int BN> struct Warps {
#ifdef BNN_EPI_WARPS
    static constexpr int EPI_WARPS = BNN_EPI_WARPS;
#else
    static constexpr int EPI_WARPS = is_f4(BN) ? 8 : 16;
#endif
    static constexpr int EPW = EPI_WARPS / 4;
    static constexpr int EPI_THREADS = EPI_WARPS * 32;
    static constexpr int MMA_WARP_B = 2 + EPI_WARPS;                 // the second MMA-issuing warp (the first is warp 1)
    static constexpr int PROD_WARP_B = MMA_WARP_B + N_ISSUE - 1;      // second producer warp (pair kernel: the B operand's loads)
    static constexpr int NTHREADS = 64 + EPI_THREADS + 32 * (N_ISSUE - 1) + 32;
};
constexpr uint32_t A_BYTES = BM * BK;
constexpr int ACC_BUFS = 2;
constexpr int ACC_MAX = 4;                      // accumulator buffers when 128-wide tiles are worked on by four epilogue teams
template <int BN> struct Cfg {
    static constexpr uint32_t B_BYTES = BN * BK;
    static constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = (BN == 256) ? 4 : (is_f4(BN) ? 5 : 6);   // 192-200 KB of operand stages
    // two accumulator buffers of BN columns; the 4-bit configuration (BN = 192) also keeps 32 columns of scale factors
    static constexpr uint32_t TMEM_COLS = is_f4(BN) ? 512 : 2 * BN;
};
constexpr int STAGES_MAX = 7;
constexpr int B_STAGES_MAX = 18;                // weight stages of the halo-tile convolution kernel (9 taps x 2 channel slices resident)

__device__ int g_umma_error;                    // 0 = fine; otherwise a code saying which wait gave up
// SM clock count and wall-clock nanoseconds at the start [0, 1] and the end [2, 3] of CTA 0 of the tensor-engine kernel that
// ran last: the clock the kernel really ran at (this part runs tensor-heavy kernels well below the maximum that
// nvidia-smi reports around them).  Two register reads and two stores by one thread per kernel.
__device__ long long g_umma_clock[4];
#define BNN_CLK_REC(i) do { if (blockIdx.x == 0 && threadIdx.x == 0) { g_umma_clock[2 * (i)] = clock64(); unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); g_umma_clock[2 * (i) + 1] = (long long)t_; } } while (0)
#ifdef BNN_TRACE
// Instrumented builds only: clock stamps of CTA 0, [role][tile][slot].
__device__ long long g_trace[8 * 16 * 16];
#define BNN_TR(role, tile, slot) do { if (blockIdx.x == 0 && (tile) < 16) g_trace[((role) * 16 + (tile)) * 16 + (slot)] = clock64(); } while (0)
#else
#define BNN_TR(role, tile, slot) do { } while (0)
#endif

struct UmmaArgs {
    int64_t M, N;
    int k_iters;            // ceil(K_bytes / BK)
    int k_last;             // MMAs (32 bytes of K each) that the last K step still needs: 1..4
    uint32_t idesc;
    int32_t *C; int64_t ldc;                     // optional int32 output
    uint32_t *out; int64_t ldo;                  // optional packed sign output
    int8_t *out8; int64_t ldo8;                  // optional +-1 output for the next layer: bytes, or
    int out_f4;                                  // ... e2m1 nibbles (two per byte, ldo8 in bytes) when set
    const int32_t *thr; const uint32_t *flip;
    // convolution mode (3x3, pad 1): A is a 4-D byte tensor [B][H][W][C_in]; one K step = (tap, 128-channel slice)
    int conv;               // 0 = plain GEMM
    int H, W, TH, TB;       // image size; a 128-pixel tile = TB images x TH rows x W columns
    int c_chunks;           // C_in / 128
    int pool;               // 2x2 max-pool (as OR of the sign bits) before the packed store
    int b_static;           // B (weights) is not written by the kernel launched just before this one
    // halo-tile convolution kernel (k_umma_conv): A stages hold a (TH + 2)-row slab of the input per horizontal tap
    int kbytes;             // k_umma_conv: bytes of channels per pixel and K step: 128 (128-byte swizzle) or 64 (64-byte swizzle)
    int a_stage_bytes, n_a_stages;   // bytes of one slab = (TH + 2) * TB * W * kbytes; slabs in the ring
    int n_b_stages;         // weight stages of BN x kbytes bytes
    int b_resident;         // all k_iters weight stages stay in shared memory (this CTA's tiles share their filters)
    int dy_bytes;           // one image row of the slab: TB * W * 128 bytes
    int tap_bytes;          // bytes of one tap in a filter row of the weight matrix (C_in bytes, or C_in / 2 for nibbles)
    int perm;               // rows of a tile are ordered (y, image, x) instead of (image, y, x)  (TB > 1)
    unsigned long long wait_ns;   // how long a wait on a barrier may last before the kernel gives up
    int drop_loads;         // test hook (single-SM kernel): the producer issues no loads, every consumer's wait runs out
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait on a phase parity.  Returns false if the limit ran out.
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2, int c3, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}
// Shared-memory matrix descriptor: K-major tile, rows of 128 bytes, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = (uint64_t)((addr & 0x3ffffu) >> 4);
    d |= (uint64_t)(1024u >> 4) << 32;   // stride byte offset
    d |= 1ull << 46;                      // descriptor version of sm_100
    d |= 2ull << 61;                      // SWIZZLE_128B
    return d;
}
// The same for rows of 64 bytes with the 64-byte swizzle: groups of eight rows 512 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw64(uint32_t addr) {
    uint64_t d = (uint64_t)((addr & 0x3ffffu) >> 4);
    d |= (uint64_t)(512u >> 4) << 32;
    d |= 1ull << 46;
    d |= 4ull << 61;                      // SWIZZLE_64B
    return d;
}
__device__ __forceinline__ void umma_i8(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// 4-bit (e2m1) operands with one UE8M0 scale per 32 values; K = 64 per instruction, float32 accumulators.
__device__ __forceinline__ void umma_mxf4(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate,
                                          uint32_t tmem_sf) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], %1, %2, %3, [%5], [%5], p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(tmem_sf) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
// Completes every tcgen05.ld issued so far.  The registers are passed through so that no use of them can be
// scheduled ahead of the wait.
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&r)[32]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
        : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
          "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]),
          "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]),
          "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
        :: "memory");
}

// Zeroes 32 accumulator columns of the calling warp's 32 lanes.  Every epilogue warp does this to the columns it has
// read (and every buffer is zeroed once at kernel start), so that every MMA of a tile ACCUMULATES: with an overwriting
// first MMA the second issuing thread had to wait at the start of every tile until that MMA had completed, and the tensor
// pipe ran on one thread's issue rate meanwhile (a pair's MMA costs its issuing thread ~120 clocks, more than the pipe
// needs to execute it): ~1200 clocks per tile.
__device__ __forceinline__ void tmem_zero32(uint32_t taddr) {
    const uint32_t z = 0u;
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1};"
                 ::"r"(taddr), "r"(z) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// All `cols` accumulator columns (a multiple of 32) of the calling warp's lane quadrant.
__device__ __forceinline__ void tmem_zero_all(uint32_t tmem_base, int warp, int cols) {
    for (int c = 0; c < cols; c += 32) tmem_zero32(tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)c);
    tmem_st_wait();
}

struct __align__(16) Control {
    uint64_t full[2 * STAGES_MAX];         // two barrier pairs per ring slot, see RingCursor
    uint64_t empty[2 * STAGES_MAX];
    uint64_t acc_full[ACC_MAX];
    uint64_t acc_empty[ACC_MAX];
    uint64_t full_b[B_STAGES_MAX];         // k_umma_conv: its weight ring (full / empty above are its slab ring); resident
    uint64_t empty_b[B_STAGES_MAX];        // weights use one pair per stage, a streamed ring two per slot
    uint32_t tmem_base;
    uint32_t failed;
    // Staged per accumulator buffer (slot s of a kernel with tiles BN wide): thresholds thr[s * BN ..] (clamped int32, or
    // float bits on the 4-bit engine) and flip words flip[s * BN / 32 ..]; 2 x 256 = 4 x 128 columns.
    __align__(16) int32_t thr[2 * BN_MAX];
    uint32_t flip[2 * BN_MAX / 32];
    // Convolution with pooling: the sign words of every pixel of a tile, [team][pixel][BN / 32 + 1] (up to two teams of
    // 256-wide tiles or four teams of 128-wide ones).
    uint32_t poolw[4 * BM * (128 / 32 + 1)];
};
static_assert(4 * BM * (128 / 32 + 1) >= 2 * BM * (BN_MAX / 32 + 1), "pooling buffer holds two teams of 256-wide tiles");

// Relaxed for the same reason as mbar_arrive_cta0 below: the barrier hands back tensor memory only.
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.relaxed.cta.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Records that a wait gave up (the first code wins): in this CTA's control block, where every other waiter of the CTA
// looks, and in the device word that bnn_device_status reads.
__device__ __forceinline__ void fail(Control *ctl, int code) {
    if (*reinterpret_cast<volatile uint32_t *>(&ctl->failed) == 0u) *reinterpret_cast<volatile uint32_t *>(&ctl->failed) = (uint32_t)code;
    atomicCAS(&g_umma_error, 0, code);
}
// Bounded wait on a phase parity: false once `limit_ns` of wall clock have passed, or as soon as another wait of this
// CTA (or of its partner in a pair) has given up, so that one failure costs one limit and not one per waiter.
__device__ __forceinline__ bool mbar_wait(const Control *ctl, unsigned long long limit_ns, uint32_t bar, uint32_t parity) {
    unsigned long long t0 = 0;
    for (uint32_t i = 0;; ++i) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
        if ((i & 63u) == 63u) {
            if (*reinterpret_cast<const volatile uint32_t *>(&ctl->failed) != 0u) return false;
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) return false;
        }
    }
}

// Position in a ring of S operand slots that is guarded by 2 S barrier pairs: stage G of a CTA's sequence lives in slot
// G % S and signals barrier pair G % 2S, phase G / 2S.
// Why twice as many barriers as slots: a wait on a phase PARITY is only right while the waiter is at most one phase ahead
// of the barrier.  Two issuing threads that take alternate stages of one ring keep that distance only when each barrier
// belongs to one of them.  With one barrier per slot and an odd S the uses of a slot alternate between the threads, and a
// thread can reach its next use while the other thread's use in between is still loading (loads complete out of
// order): the parity it waits for then matches the phase before, the wait returns at once, and it multiplies a slot
// that is being written and releases it a second time.  2 S is even, so every barrier pair has one consumer thread.
struct RingCursor {
    uint32_t b, lap;                 // barrier pair of the next stage; how often the barrier ring has wrapped
    // M: barrier pairs per slot (2 for two consumer threads that alternate; a multiple of the number of threads that
    // take the stages in turn, so that G % (M S) fixes the thread)
    __host__ __device__ __forceinline__ void start(uint32_t G, uint32_t S, uint32_t M = 2) { b = G % (M * S); lap = G / (M * S); }
    __host__ __device__ __forceinline__ uint32_t slot(uint32_t S) const { uint32_t x = b; while (x >= S) x -= S; return x; }
    __host__ __device__ __forceinline__ uint32_t parity() const { return lap & 1u; }
    // the stage that used this slot before (S stages earlier): whether there is one, its barrier pair and phase parity
    __host__ __device__ __forceinline__ bool reuses(uint32_t S) const { return lap > 0 || b >= S; }
    __host__ __device__ __forceinline__ uint32_t prev_bar(uint32_t S, uint32_t M = 2) const { return b >= S ? b - S : b + (M - 1) * S; }
    __host__ __device__ __forceinline__ uint32_t prev_parity(uint32_t S) const { return (b >= S ? lap : lap - 1u) & 1u; }
    __host__ __device__ __forceinline__ void advance(uint32_t n, uint32_t S, uint32_t M = 2) { b += n; if (b >= M * S) { b -= M * S; ++lap; } }   // n <= M S
};

// 8 sign bits -> 8 e2m1 nibbles (+1.0 = 0x2, -1.0 = 0xa); bit i lands in nibble i.
__device__ __forceinline__ uint32_t nibbles_of_byte(uint32_t x) {
    // bit pairs -> selector nibbles 0..3, then one byte permute out of the four possible nibble pairs
    uint32_t t = (x | (x << 4)) & 0x0f0fu;
    t = (t | (t << 2)) & 0x3333u;
    return __byte_perm(0x222aa2aau, 0u, t);       // pair 00 -> 0xaa, 01 -> 0xa2, 10 -> 0x2a, 11 -> 0x22
}
// The signs of 32 consecutive outputs of row `orow` (bit j of `word` = column col0 + j) in the next layer's operand
// format: one signed byte per value, or one e2m1 nibble per value.  Positions at or beyond N are written as 0.
// role / hold (nibble output): a warp that takes two adjacent 32-column chunks keeps the first chunk's 16 bytes (role 1)
// and writes both with one 32-byte store when it has the second (role 2): whole sectors instead of half ones.
__device__ __forceinline__ void store_signs(const UmmaArgs &p, uint32_t word, int64_t orow, int64_t col0, int role = 0,
                                            uint4 *hold = nullptr) {
    if (p.out_f4) {
        uint8_t *d = reinterpret_cast<uint8_t *>(p.out8) + orow * p.ldo8 + (col0 >> 1);
        if (role != 0) {
            // both chunks whole, and the pair's 32 bytes on a 32-byte boundary (the same answer in both roles)
            const int64_t first = (role == 1) ? col0 : col0 - 32;
            uint8_t *d0 = reinterpret_cast<uint8_t *>(p.out8) + orow * p.ldo8 + (first >> 1);
            if (first + 64 <= p.N && (reinterpret_cast<uintptr_t>(d0) & 31u) == 0) {
                const uint4 v = make_uint4(nibbles_of_byte(word & 0xffu), nibbles_of_byte((word >> 8) & 0xffu),
                                           nibbles_of_byte((word >> 16) & 0xffu), nibbles_of_byte(word >> 24));
                if (role == 1) { *hold = v; return; }
                asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                             ::"l"(d0), "r"(hold->x), "r"(hold->y), "r"(hold->z), "r"(hold->w), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
                return;
            }
        }
        if (col0 + 32 <= p.N) {
            *reinterpret_cast<uint4 *>(d) = make_uint4(nibbles_of_byte(word & 0xffu), nibbles_of_byte((word >> 8) & 0xffu),
                                                       nibbles_of_byte((word >> 16) & 0xffu), nibbles_of_byte(word >> 24));
        } else {
            for (int j = 0; j < 32; j += 2) {
                if ((col0 + j) / 2 >= p.ldo8) break;
                const uint32_t lo = (col0 + j < p.N) ? (((word >> j) & 1u) ? 0x2u : 0xau) : 0u;
                const uint32_t hi = (col0 + j + 1 < p.N) ? (((word >> (j + 1)) & 1u) ? 0x2u : 0xau) : 0u;
                d[j >> 1] = (uint8_t)(lo | (hi << 4));
            }
        }
        return;
    }
    int8_t *d8 = p.out8 + orow * p.ldo8 + col0;
    if (col0 + 32 <= p.N) {
        uint32_t b[8];
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            // 4 sign bits -> 4 bytes of +1 (0x01) / -1 (0xff)
            const uint32_t t4 = (((word >> (4 * g)) & 0xfu) * 0x00204081u) & 0x01010101u;
            b[g] = ~(t4 * 0xfeu);
        }
        if ((reinterpret_cast<uintptr_t>(d8) & 31u) == 0) {   // one 256-bit store: a whole 32-byte sector per thread
            asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                         ::"l"(d8), "r"(b[0]), "r"(b[1]), "r"(b[2]), "r"(b[3]), "r"(b[4]), "r"(b[5]), "r"(b[6]), "r"(b[7]) : "memory");
        } else {
            *reinterpret_cast<uint4 *>(d8) = make_uint4(b[0], b[1], b[2], b[3]);
            *reinterpret_cast<uint4 *>(d8 + 16) = make_uint4(b[4], b[5], b[6], b[7]);
        }
    } else {
        for (int j = 0; j < 32; ++j)
            if (col0 + j < p.N) d8[j] = ((word >> j) & 1u) ? (int8_t)1 : (int8_t)-1;
            else if (col0 + j < p.ldo8) d8[j] = 0;
    }
}

// One 32-column chunk of accumulators (r, one output row per thread) -> the requested outputs.
template <int BN, bool F4 = is_f4(BN)>
__device__ __forceinline__ void epilogue_chunk(Control *ctl, const UmmaArgs &p, uint32_t (&r)[32], uint32_t buf, int c, int64_t col0,
                                               int64_t row, int lin, uint32_t *poolw, int role = 0, uint4 *hold = nullptr) {
    // buf: the slot whose staged thresholds apply; poolw: this team's pooling buffer, BN / 32 + 1 words per pixel
    if (row >= p.M) return;
    if (p.thr) {                                         // thresholded signs: packed words and/or the next layer's operand
        // bit j of the word = (acc[j] >= thr[j]) = NOT sign(acc[j] - thr[j]); the sign bits are shifted
        // into four independent 8-bit chains (funnel shift: one instruction per column after the subtract)
        const int4 *tp = reinterpret_cast<const int4 *>(&ctl->thr[buf * BN + 32 * c]);
        uint32_t w4[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int g = 7; g >= 0; --g) {
            const int4 t = tp[g];
            const int tv[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
            for (int i = 3; i >= 0; --i) {
                const int j = 4 * g + i;
                const uint32_t d = F4 ? __float_as_uint(__uint_as_float(r[j]) - __int_as_float(tv[i]))
                                               : (uint32_t)((int32_t)r[j] - tv[i]);
                w4[j >> 3] = __funnelshift_l(d, w4[j >> 3], 1);
            }
        }
        const uint32_t lt = __byte_perm(__byte_perm(w4[0], w4[1], 0x0040), __byte_perm(w4[2], w4[3], 0x0040), 0x5410);
        const uint32_t flipw = ctl->flip[buf * (BN / 32) + c];
        uint32_t word = ~lt ^ flipw;
        if (col0 + 32 > p.N) word &= (1u << (p.N - col0)) - 1u;      // columns beyond N stay 0
        if (p.pool) poolw[lin * (BN / 32 + 1) + c] = word ^ flipw;   // un-flipped (dot >= thr) bits
        else if (p.out) p.out[row * p.ldo + (col0 >> 5)] = word;
        if (p.out8 && !p.pool) store_signs(p, word, row, col0, role, hold);
    }
    if (p.C) {
        if (F4) {   // the 4-bit engine accumulates in float32: exact integers
            if (p.k_iters <= (1 << 14)) {
                // |sum| <= K <= 2^22: adding 1.5 * 2^23 leaves the integer in the low mantissa bits (an add and a
                // subtract on the full-rate pipes instead of a quarter-rate conversion)
#pragma unroll
                for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + 12582912.0f) - 0x4b400000u;
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) r[j] = (uint32_t)(int32_t)__uint_as_float(r[j]);
            }
        }
        int32_t *dst = p.C + row * p.ldc + col0;
        if (col0 + 32 <= p.N && ((reinterpret_cast<uintptr_t>(dst) & 31u) == 0)) {
            // 256-bit stores: whole 32-byte sectors, four instructions for the thread's 128 bytes; streamed, because the
            // sums are not re-read while the operands are
#pragma unroll
            for (int j = 0; j < 32; j += 8)
                asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                             ::"l"(dst + j), "r"(r[j]), "r"(r[j + 1]), "r"(r[j + 2]), "r"(r[j + 3]), "r"(r[j + 4]), "r"(r[j + 5]),
                               "r"(r[j + 6]), "r"(r[j + 7]) : "memory");
        } else if (col0 + 32 <= p.N && ((reinterpret_cast<uintptr_t>(dst) & 15u) == 0)) {
#pragma unroll
            for (int j = 0; j < 32; j += 4)
                __stcs(reinterpret_cast<int4 *>(dst + j), make_int4((int)r[j], (int)r[j + 1], (int)r[j + 2], (int)r[j + 3]));   // streamed: the sums are not re-read, the operands are
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (col0 + j < p.N) dst[j] = (int32_t)r[j];
        }
    }
}

// One tile's epilogue for the calling epilogue warp: stage the tile's thresholds, wait for the accumulators in
// buffer `buf`, and turn them into the requested outputs.  `ok` turns false once a wait has given up.
// The staged form of a threshold.  The comparison is the sign of (accumulator - threshold); accumulators stay below 2^30
// in magnitude (2^24 on the 4-bit engine, where they are float32), so thresholds clamp to that range unchanged in meaning.
template <bool F4>
__device__ __forceinline__ int32_t staged_threshold(int32_t t) {
    if (F4) return __float_as_int(t > (1 << 24) ? 3.0e7f : (t < -(1 << 24) ? -3.0e7f : (float)t));
    return max(min(t, 1 << 30), -(1 << 30));
}

// n0_next: first column of the tile this CTA handles next (-1: none).  Its thresholds are fetched from global memory
// while this tile is processed and staged for the other buffer at the end, so no tile but the first waits for them.
// Row i of a convolution tile -> the pixel's position in (image, y, x) order inside the tile.  The halo-tile kernel keeps
// tiles of several small images in (y, image, x) order, so that one tap's rows are evenly spaced in shared memory.
__device__ __forceinline__ int tile_lin(const UmmaArgs &p, int i) {
    if (!p.perm) return i;
    const int x = i % p.W, b = (i / p.W) % p.TB, y = i / (p.W * p.TB);
    return (b * p.TH + y) * p.W + x;
}

// EPI_WARPS: the warps that work on this tile together.  A kernel may run several such teams (TEAM = 0 .. 3) on different
// tiles at once, each with its own pooling buffer and pair of named barriers.  buf = the accumulator buffer (and slot of
// staged thresholds) of this tile, acc_parity the phase of its "full" barrier, slot_next the slot that receives the
// thresholds of the team's next tile (first column n0_next; -1 = none; same_next = they are the ones already staged);
// `first` says that this is the team's first tile (it stages its own thresholds).
template <int BN, bool F4 = is_f4(BN), int EPI_WARPS = Warps<BN>::EPI_WARPS, int TEAM = 0, bool PREFETCH = true>
__device__ __forceinline__ void epilogue_tile(Control *ctl, const UmmaArgs &p, uint32_t tmem_base, uint32_t buf, uint32_t tc,
                                              int64_t m0, int64_t n0, int64_t n0_next, int q, int half, int lane, int et, bool &ok,
                                              bool first, uint32_t acc_parity, uint32_t slot_next, bool same_next = false) {
    constexpr int EPW = EPI_WARPS / 4, EPI_THREADS = EPI_WARPS * 32;
    constexpr int BAR_A = 1 + 2 * TEAM, BAR_B = 2 + 2 * TEAM;      // named barriers of this team
    uint32_t *poolw = ctl->poolw + TEAM * BM * (BN / 32 + 1);
    static_assert(BN <= EPI_THREADS, "one staged threshold per epilogue thread");
    constexpr int CHUNKS = BN / 32, CPW = (CHUNKS + 1) / 2;   // 32-column chunks per tile and (at most) per warp with two warps per quadrant
    const int lin = tile_lin(p, 32 * q + lane);
    const int64_t row = m0 + lin;
    if (p.thr && first) {                                // the first tile stages its own thresholds
        if (et < BN) ctl->thr[buf * BN + et] = staged_threshold<F4>((n0 + et < p.N) ? p.thr[n0 + et] : 0x7fffffff);
        if (et < BN / 32) {
            const int64_t w = (n0 >> 5) + et;
            ctl->flip[buf * (BN / 32) + et] = (p.flip && w * 32 < p.N) ? p.flip[w] : 0u;
        }
    }
    const int tr_role = (et == 0) ? 3 : ((et == EPI_THREADS - 32) ? 4 : -1);
    if (tr_role >= 0) BNN_TR(tr_role, tc, 0);
    if (tr_role >= 0) BNN_TR(tr_role, tc, 1);
    const bool have_next = p.thr && n0_next >= 0 && !same_next;      // (same_next: the thresholds already staged stay valid)
    int32_t next_thr = 0x7fffffff;
    uint32_t next_flip = 0u;
    if (have_next) {
        if (et < BN && n0_next + et < p.N) next_thr = p.thr[n0_next + et];
        if (et < BN / 32) {
            const int64_t w = (n0_next >> 5) + et;
            if (p.flip && w * 32 < p.N) next_flip = p.flip[w];
        }
    }
    // One warp polls the "accumulator full" barrier; the others park on a hardware barrier until it has seen it.  A
    // polling warp takes an issue slot on every turn of its loop, and with four of them on each scheduler the two
    // MMA-issuing threads, which share those schedulers, needed three times as long per instruction: a tile of nine
    // short K steps then ran at 40 % of the tensor pipe's rate.
    if (et < 32 && ok && !mbar_wait(ctl, p.wait_ns, smem_u32(&ctl->acc_full[buf]), acc_parity)) { fail(ctl, 3); ok = false; }
    // (the same barrier makes the staged thresholds visible and says that nobody reads the previous tile's pooling words)
    asm volatile("bar.sync %0, %1;" ::"n"(BAR_B), "n"(EPI_THREADS) : "memory");
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (tr_role >= 0) BNN_TR(tr_role, tc, 2);
    ok = ok && (ctl->failed == 0);
    if (ok) {
        const uint32_t tbase = tmem_base + ((uint32_t)(32 * q) << 16) + buf * BN;
        if constexpr (EPW == 2 && PREFETCH) {
            // two warps per quadrant, each a contiguous half of the columns (the first one chunk more when their number
            // is odd): chunk c+1 is fetched from tensor memory while chunk c is processed (unrolled, so both register
            // buffers are addressed statically)
            uint32_t ra[32], rb[32];
            const int c_first = half * CPW, c_end = half ? CHUNKS : CPW;
            if (n0 + 32 * c_first < p.N) { tmem_ld32(tbase + (uint32_t)(32 * c_first), ra); tmem_ld_wait(ra); tmem_zero32(tbase + (uint32_t)(32 * c_first)); }
#pragma unroll
            for (int cc = 0; cc < CPW; ++cc) {
                const int c = c_first + cc;
                const int64_t col0 = n0 + 32 * c;
                if (c >= c_end || col0 >= p.N) break;        // uniform over the warp
                const bool more = (c + 1 < c_end) && (col0 + 32 < p.N);
                uint32_t (&r)[32] = (cc & 1) ? rb : ra;
                uint32_t (&rn)[32] = (cc & 1) ? ra : rb;
                if (more) tmem_ld32(tbase + (uint32_t)(32 * (c + 1)), rn);
                epilogue_chunk<BN, F4>(ctl, p, r, buf, c, col0, row, lin, poolw);
                if (more) { tmem_ld_wait(rn); tmem_zero32(tbase + (uint32_t)(32 * (c + 1))); }
            }
        } else {
            // more warps per quadrant: chunks go round-robin over them, one register buffer, and the other warps of
            // the scheduler cover the load latency
            uint32_t r[32];
            if constexpr (EPW == 2) {
                // two warps per quadrant, each a contiguous half of the columns, one chunk at a time (kernels whose thread
                // count leaves no registers for a second chunk in flight); adjacent chunks pair up for whole-sector stores
                const int c_first = half * CPW, c_end = half ? CHUNKS : CPW;
                uint4 hold = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll 1
                for (int c = c_first; c < c_end; ++c) {
                    const int64_t col0 = n0 + 32 * c;
                    if (col0 >= p.N) break;                  // uniform over the warp
                    tmem_ld32(tbase + (uint32_t)(32 * c), r);
                    tmem_ld_wait(r);
                    tmem_zero32(tbase + (uint32_t)(32 * c));
                    const int role = (CPW % 2 == 0) ? 1 + ((c - c_first) & 1) : 0;
                    epilogue_chunk<BN, F4>(ctl, p, r, buf, c, col0, row, lin, poolw, role, &hold);
                }
            } else if constexpr (CHUNKS == 2 * EPW) {
                // two adjacent chunks per warp, so that nibble outputs leave as whole 32-byte sectors
                uint4 hold = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll 1
                for (int i = 0; i < 2; ++i) {
                    const int c = 2 * half + i;
                    const int64_t col0 = n0 + 32 * c;
                    if (col0 >= p.N) break;                  // uniform over the warp
                    tmem_ld32(tbase + (uint32_t)(32 * c), r);
                    tmem_ld_wait(r);
                    tmem_zero32(tbase + (uint32_t)(32 * c));
                    epilogue_chunk<BN, F4>(ctl, p, r, buf, c, col0, row, lin, poolw, 1 + i, &hold);
                }
            } else {
                uint4 hold = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll 1
                for (int c = half; c < CHUNKS; c += EPW) {
                    const int64_t col0 = n0 + 32 * c;
                    if (col0 >= p.N) break;                  // uniform over the warp
                    tmem_ld32(tbase + (uint32_t)(32 * c), r);
                    tmem_ld_wait(r);
                    tmem_zero32(tbase + (uint32_t)(32 * c));
                    // one warp per quadrant walks all chunks: adjacent ones pair up for whole-sector nibble stores
                    const int role = (EPW == 1 && CHUNKS % 2 == 0) ? 1 + (c & 1) : 0;
                    epilogue_chunk<BN, F4>(ctl, p, r, buf, c, col0, row, lin, poolw, role, &hold);
                }
            }
        }
        tmem_st_wait();                                  // the zeroes are in place before the buffer is handed back
        // padding words of the packed output
        if (half == 0 && p.out && !p.pool && row < p.M && n0 + BN >= p.N) {
            for (int64_t w = (p.N + 31) >> 5; w < p.ldo; ++w) p.out[row * p.ldo + w] = 0u;
        }
    }
    if (tr_role >= 0) BNN_TR(tr_role, tc, 3);
    if (p.pool) {
        // 2x2 max-pool then threshold == OR of the four thresholded bits, then flip.  The tile holds TB images
        // x TH rows x W columns (TH, W even), i.e. 32 whole windows; 256 (window, word) items for 128 threads.
        asm volatile("bar.sync %0, %1;" ::"n"(BAR_A), "n"(EPI_THREADS) : "memory");
        if (ok) {
            const int Wo = p.W >> 1, nwords = (int)((min((int64_t)BN, p.N - n0) + 31) >> 5);
            for (int e = et; e < (BM / 4) * (BN / 32); e += EPI_THREADS) {
                const int win = e / (BN / 32), c = e % (BN / 32);
                if (c >= nwords) continue;
                const int wx = win % Wo, wy = win / Wo;                 // wy counts window rows over the tile's TB*TH/2 rows
                const int r0 = (2 * wy) * p.W + 2 * wx;                 // top-left pixel of the window inside the tile
                const int64_t pix = m0 + r0;                            // its linear pixel index b*H*W + y*W + x
                if (pix >= p.M) continue;
                constexpr int PP = BN / 32 + 1;
                uint32_t word = poolw[r0 * PP + c] | poolw[(r0 + 1) * PP + c] | poolw[(r0 + p.W) * PP + c] | poolw[(r0 + p.W + 1) * PP + c];
                word ^= ctl->flip[buf * (BN / 32) + c];
                const int64_t col0 = n0 + 32 * c;
                if (col0 + 32 > p.N) word &= (1u << (p.N - col0)) - 1u;
                // output pixel: same image, (y/2, x/2).  The tile starts at x = 0 of an even row and holds whole rows (of
                // one image or of TB whole images), so its 32 windows are 32 consecutive output pixels from m0 / 4 on.
                const int64_t opix = (m0 >> 2) + win;
                p.out[opix * p.ldo + (col0 >> 5)] = word;
                if (n0 + BN >= p.N && c == nwords - 1)
                    for (int64_t w = (p.N + 31) >> 5; w < p.ldo; ++w) p.out[opix * p.ldo + w] = 0u;
                if (p.out8) store_signs(p, word, opix, col0);   // the pooled pixel's signs for the next layer
            }
        }
    }
    if (tr_role >= 0) BNN_TR(tr_role, tc, 4);
    if (have_next) {
        // (a team that stays on one accumulator buffer restages that buffer's thresholds: only when all have finished reading)
        if (slot_next == buf) asm volatile("bar.sync %0, %1;" ::"n"(BAR_A), "n"(EPI_THREADS) : "memory");
        // Every epilogue thread has passed this tile's barrier, so none still reads the other buffer's thresholds (they
        // belonged to the previous tile); the next tile's barrier makes these visible.
        if (et < BN) ctl->thr[slot_next * BN + et] = staged_threshold<F4>(next_thr);
        if (et < BN / 32) ctl->flip[slot_next * (BN / 32) + et] = next_flip;
    }
    if (tr_role >= 0) BNN_TR(tr_role, tc, 5);
}

// Persistent: gridDim.x CTAs (one per SM) walk the tile list with stride gridDim.x.  The shared-memory ring
// runs on across tiles; the accumulator is double-buffered in tensor memory (2 x 256 columns), so the
// epilogue of tile i overlaps the main loop of tile i+1.
// TEAMS > 1: the epilogue warps form that many teams, team k on the CTA's tiles k, k + TEAMS, ... with an accumulator
// buffer of its own (TEAMS x BN columns of tensor memory).  For tiles with few K steps the epilogue, ~2500 clocks of
// mostly latency per tile, is what the tile rate follows; with several tiles' epilogues in flight it is their throughput.
template <int BN, int TEAMS = 1>
__global__ void __launch_bounds__(Warps<BN>::NTHREADS, 1)
k_umma_i8(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, const UmmaArgs p) {
    constexpr int STAGES = Cfg<BN>::STAGES;
    constexpr uint32_t STAGE_BYTES = Cfg<BN>::STAGE_BYTES;
    constexpr int EPI_WARPS = Warps<BN>::EPI_WARPS, MMA_WARP_B = Warps<BN>::MMA_WARP_B;
    constexpr int NBUF = TEAMS == 1 ? ACC_BUFS : TEAMS, TW = EPI_WARPS / TEAMS;      // accumulator buffers; warps per team
    static_assert(TEAMS == 1 || (!is_f4(BN) && NBUF * BN <= 512 && TW % 4 == 0), "teams: byte tiles whose buffers fit tensor memory");
    constexpr uint32_t TMEM_COLS = TEAMS == 1 ? Cfg<BN>::TMEM_COLS : (NBUF * BN <= 256 ? 256 : 512);
    extern __shared__ uint8_t smem_raw[];
    // operand tiles need 1024-byte alignment for the 128-byte swizzle pattern
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Control *ctl = reinterpret_cast<Control *>(tiles + STAGES * STAGE_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t tiles_m = (p.M + BM - 1) / BM;
    const int64_t tiles_n = (p.N + BN - 1) / BN;
    const int64_t ntiles = tiles_m * tiles_n;
    BNN_CLK_REC(0);

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2 * STAGES; ++s) { mbar_init(smem_u32(&ctl->full[s]), 1); mbar_init(smem_u32(&ctl->empty[s]), 1); }
        for (int b = 0; b < NBUF; ++b) {
            mbar_init(smem_u32(&ctl->acc_full[b]), N_ISSUE);    // one commit from each MMA-issuing warp
            mbar_init(smem_u32(&ctl->acc_empty[b]), TW);        // the warps of the team that reads this buffer
        }
        ctl->failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = ctl->tmem_base;
    // Barriers and tensor memory were set up while the preceding kernel drained; what reads or writes global memory
    // waits for it below (bnn_pdl_wait): the producer (after requesting weights that kernel does not write), the
    // epilogue warps at once; they also release this kernel's own successor.

    {
        // Every accumulator buffer starts at zero (all MMAs accumulate, see tmem_zero32).
        // 4-bit engine: every value is exactly +-1, so every block scale is 2^0.  In UE8M0 that is the byte 0x7f, and
        // with all 32 scale-factor columns filled with it the instruction reads 1.0 wherever it looks.
        if (warp >= 2 && warp < 6) {
            tmem_zero_all(tmem_base, warp, NBUF * BN);
            if (is_f4(BN)) {
                const uint32_t v = 0x7f7f7f7fu;
                asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1};"
                             ::"r"(tmem_base + SF_COL + ((uint32_t)(32 * (warp & 3)) << 16)), "r"(v) : "memory");
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    }

    if (warp == 0) {
        // ---------------- TMA producer (with the test hook set it requests nothing: every consumer's wait runs out)
        if (lane == 0 && !p.drop_loads) {
            bool ok = true;
            // The loop below runs once per K step in a single thread that shares its scheduler with epilogue warps:
            // everything per tile is computed once, ring slot / phase / tap advance incrementally (no divisions inside;
            // with them a 3x3 convolution's producer could not keep up: 128 -> 128 channels at 32 x 32, 88 -> 57 us).
            RingCursor rc; rc.start(0, STAGES);
            const uint32_t tn32 = (uint32_t)tiles_n;
            // B is weights, not a product of the preceding kernel: its share of the first ring fill is requested before
            // the wait for that kernel, A's after it
            const int npre = !p.b_static ? 0 : (p.k_iters < STAGES ? p.k_iters : STAGES);
            {
                const int n0f = (int)((blockIdx.x % tn32) * BN);
                for (int kit = 0; kit < npre; ++kit) {
                    const uint32_t bar = smem_u32(&ctl->full[kit]);
                    mbar_expect_tx(bar, STAGE_BYTES);
                    tma_load_2d(smem_u32(tiles + kit * STAGE_BYTES + A_BYTES), &mapB, kit * BK, n0f, bar);
                }
            }
            bnn_pdl_wait();
            for (uint32_t t = blockIdx.x; t < (uint32_t)ntiles && ok; t += gridDim.x) {
                const bool first_tile = (t == blockIdx.x);
                const uint32_t tm = t / tn32;
                const int m0 = (int)(tm * BM), n0 = (int)((t - tm * tn32) * BN);
                int b0 = 0, y0 = 0;
                if (p.conv) {
                    // tile -> (first image, first row); K step -> (tap, channel slice); halo rows/columns and
                    // images beyond the batch are outside the tensor and arrive as zeros
                    const int tiles_per_img = p.H / p.TH;
                    b0 = (p.TB > 1) ? (int)tm * p.TB : (int)tm / tiles_per_img;
                    y0 = (p.TB > 1) ? 0 : ((int)tm % tiles_per_img) * p.TH;
                }
                int cc = 0, tx = -1, ty = -1;            // channel slice and tap offsets of the current K step
                for (int kit = 0; kit < p.k_iters; ++kit) {
                    const bool pre = first_tile && kit < npre;      // B already requested, bytes already expected
                    if (kit == 0) BNN_TR(0, (t - blockIdx.x) / gridDim.x, 0);
                    if (rc.reuses(STAGES) && !mbar_wait(ctl, p.wait_ns, smem_u32(&ctl->empty[rc.prev_bar(STAGES)]), rc.prev_parity(STAGES))) { fail(ctl, 1); ok = false; break; }
                    if (kit == 0) BNN_TR(0, (t - blockIdx.x) / gridDim.x, 1);
                    const uint32_t bar = smem_u32(&ctl->full[rc.b]);
                    if (!pre) mbar_expect_tx(bar, STAGE_BYTES);
                    const uint32_t dst = smem_u32(tiles + rc.slot(STAGES) * STAGE_BYTES);
                    if (p.conv) {
                        tma_load_4d(dst, &mapA, cc * BK, tx, y0 + ty, b0, bar);
                        if (++cc == p.c_chunks) { cc = 0; if (++tx == 2) { tx = -1; ++ty; } }
                    } else {
                        tma_load_2d(dst, &mapA, kit * BK, m0, bar);
                    }
                    if (!pre) tma_load_2d(dst + A_BYTES, &mapB, kit * BK, n0, bar);
                    rc.advance(1, STAGES);
                }
            }
        }
    } else if (warp == 1 || warp == MMA_WARP_B) {
        // ---------------- MMA issuers.  Issuing one K step (wait, four instructions, commit) costs the issuing thread
        // more clocks than the tensor core needs to execute it, so N_ISSUE warps on different schedulers share the work
        // round-robin over the K steps of every tile.  All products are exact integers and every MMA accumulates into a
        // buffer that the epilogue left at zero, so the order in which the streams reach the accumulator does not matter.
        if (lane == 0) {
            const int w = (warp == 1) ? 0 : warp - MMA_WARP_B + 1;   // this warp takes K steps w, w + N_ISSUE, ...
            // e2m1 x e2m1 (format 1), UE8M0 scales (bit 23) on the 4-bit engine; N >> 3 at bit 17, M >> 4 at bit 24
            const uint32_t idesc = is_f4(BN)
                ? ((1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | (1u << 23) | ((uint32_t)(BM >> 4) << 24))
                : (p.idesc | ((uint32_t)(BN >> 3) << 17));
            const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
            const uint64_t adesc0 = smem_desc_sw128(smem_u32(tiles)), bdesc0 = smem_desc_sw128(smem_u32(tiles + A_BYTES));
            uint32_t it0 = 0, tc = 0;                    // it0: K steps of this CTA before the current tile
            bool ok = true;
            for (int64_t t = blockIdx.x; t < ntiles && ok; t += gridDim.x, ++tc, it0 += (uint32_t)p.k_iters) {
                const uint32_t buf = tc % NBUF, use = tc / NBUF;
                if (use > 0 && !mbar_wait(ctl, p.wait_ns, smem_u32(&ctl->acc_empty[buf]), (use - 1) & 1)) { fail(ctl, 4); ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                BNN_TR(1 + w, tc, 0);
                const uint32_t tmem_d = tmem_base + buf * BN;
                RingCursor rc; rc.start(it0 + w, STAGES);            // this warp's next step
                for (int kit = w; kit < p.k_iters; kit += N_ISSUE) {
                    if (!mbar_wait(ctl, p.wait_ns, full0 + 8 * rc.b, rc.parity())) { fail(ctl, 2); ok = false; break; }
                    const uint32_t s = rc.slot(STAGES);
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    if (kit < 2) BNN_TR(1 + w, tc, 1 + kit);
                    const uint64_t adesc = adesc0 + (uint64_t)(s * (STAGE_BYTES >> 4));
                    const uint64_t bdesc = bdesc0 + (uint64_t)(s * (STAGE_BYTES >> 4));
                    const int nk = (kit == p.k_iters - 1) ? p.k_last : BK / 32;   // the last step may end early (K not a multiple of BK)
#pragma unroll
                    for (int k = 0; k < BK / 32; ++k) {   // 32 bytes of K per instruction: start address advances by 32 B (>> 4 = 2)
                        if (k >= nk) break;
                        if (is_f4(BN)) umma_mxf4(tmem_d, adesc + 2 * k, bdesc + 2 * k, idesc, 1u, tmem_base + SF_COL);
                        else umma_i8(tmem_d, adesc + 2 * k, bdesc + 2 * k, idesc, 1u);
                    }
                    umma_commit(empty0 + 8 * rc.b);             // stage may be refilled once these MMAs have read it
                    rc.advance(N_ISSUE, STAGES);
                }
                umma_commit(smem_u32(&ctl->acc_full[buf]));     // this warp's share of the tile complete (also after a failure)
                BNN_TR(1 + w, tc, 11);
            }
        }
    } else if (warp < 2 + EPI_WARPS) {
        // ---------------- epilogue: warps 2..9; warp w may only touch TMEM lanes 32*(w%4) .. +31, so two warps share
        // each lane quadrant and split the tile's columns between them
        bnn_pdl_wait();
        bnn_pdl_launch_next();
        const int q = warp & 3;
        const int team = (warp - 2) / TW;
        const int half = ((warp - 2) % TW) >> 2;
        const int et = (threadIdx.x - 64) % (32 * TW);   // 0 .. 32 * TW - 1 among the team's threads
        bool ok = true;
        // 32-bit tile arithmetic (the host checks the tile count)
        const uint32_t tn = (uint32_t)tiles_n, nt = (uint32_t)ntiles;
        for (uint32_t tc = (uint32_t)team; ; tc += TEAMS) {
            const uint32_t t = blockIdx.x + tc * gridDim.x;
            if (t >= nt) break;
            const uint32_t tm_i = t / tn;
            const int64_t m0 = (int64_t)tm_i * BM, n0 = (int64_t)(t - tm_i * tn) * BN;
            const uint32_t t2 = t + TEAMS * gridDim.x;
            const int64_t n0_next = (t2 < nt) ? (int64_t)(t2 % tn) * BN : -1;
            uint32_t buf;
            if constexpr (TEAMS == 1) {
                buf = tc & 1;
                epilogue_tile<BN>(ctl, p, tmem_base, buf, tc, m0, n0, n0_next, q, half, lane, et, ok, tc == 0, (tc / ACC_BUFS) & 1, buf ^ 1u);
            } else {
                buf = (uint32_t)team;
                const bool first = tc < (uint32_t)TEAMS, same = n0_next == n0;
                const uint32_t par = (tc / TEAMS) & 1u;
#define BNN_EPI_TEAM(K) epilogue_tile<BN, false, TW, K, false>(ctl, p, tmem_base, buf, tc, m0, n0, n0_next, q, half, lane, et, ok, first, par, buf, same)
                if (TEAMS > 3 && team == 3) BNN_EPI_TEAM((TEAMS > 3 ? 3 : 0));
                else if (TEAMS > 2 && team == 2) BNN_EPI_TEAM((TEAMS > 2 ? 2 : 0));
                else if (team == 1) BNN_EPI_TEAM(1);
                else BNN_EPI_TEAM(0);
#undef BNN_EPI_TEAM
            }
            // hand the accumulator buffer back to the MMA warp
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[buf]));
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    BNN_CLK_REC(1);
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------------------
// Two-SM variant (GEMM mode): a cluster of two CTAs computes a 256 x 256 tile with tcgen05.mma cta_group::2.
// Each CTA loads its own 128 rows of A and its own 128 of the tile's 256 B rows (32 KB per K step instead of
// 48 KB, six stages), so the L2 -> shared-memory traffic per MAC drops by a third; the pair's tensor cores read
// both halves of B.  CTA 0 of the pair issues the MMAs; completion of every CTA's TMA loads is counted on CTA 0's
// "full" barrier, stages and accumulators are released to both CTAs with multicast tcgen05.commit, and the
// epilogue warps of both CTAs hand their accumulator buffer back by arriving on CTA 0's barrier.
template <int BN> struct Cfg2 {
    static constexpr uint32_t STAGE_BYTES = A_BYTES + (BN / 2) * BK;    // own A rows + own half of the tile's B rows
    static constexpr int STAGES = (BN == 256) ? 6 : 7;                  // 192 / 196 KB
};
constexpr uint32_t PEER_MASK = 0xFEFFFFFFu;              // clears the CTA-rank bit of a shared::cluster address -> CTA 0 of the pair

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d_2sm(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_4d_2sm(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2, int c3, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}
__device__ __forceinline__ void umma_i8_2sm(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives on the barrier at this shared-memory offset in both CTAs of the pair once the MMAs issued so far are done.
__device__ __forceinline__ void umma_commit_2sm(uint32_t bar) {
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}
// Arrive on the barrier at the same offset in CTA 0 of the cluster.  Relaxed: the barrier hands back tensor memory, whose
// reads are ordered by tcgen05.wait::ld and the tcgen05 fence before the arrival; nothing written to memory is passed
// on through it.  (With release semantics at cluster scope the arrival waited for the epilogue's global stores to
// complete: ~3800 clocks per tile, during which the issuing warps could not reuse the accumulator buffer.)
__device__ __forceinline__ void mbar_arrive_cta0(uint32_t bar) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, 0;" : "=r"(remote) : "r"(bar));
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}

// A failed wait in one CTA of a pair: recorded locally (fail) and in the partner's control block, so that the partner's
// waiters stop at their next look instead of each running into the limit.  Both CTAs stay resident until the
// cluster-wide barrier at the end of the kernel, so the partner's shared memory is there to be written.
__device__ __forceinline__ void fail_pair(Control *ctl, int code) {
    fail(ctl, code);
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(&ctl->failed)), "r"(cluster_ctarank() ^ 1u));
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(remote), "r"((uint32_t)code) : "memory");
}

// 4-bit form of the pair instruction (see umma_mxf4).
__device__ __forceinline__ void umma_mxf4_2sm(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate,
                                              uint32_t tmem_sf) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::mxf4.block_scale.block32 [%0], %1, %2, %3, [%5], [%5], p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(tmem_sf) : "memory");
}

template <int BN, int TEAMS = 1>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(Warps<BN>::NTHREADS, 1)
k_umma_i8_2sm(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, const UmmaArgs p) {
    constexpr int STAGES2 = Cfg2<BN>::STAGES;
    constexpr uint32_t STAGE2_BYTES = Cfg2<BN>::STAGE_BYTES;
    constexpr int EPI_WARPS = Warps<BN>::EPI_WARPS, MMA_WARP_B = Warps<BN>::MMA_WARP_B;
    constexpr int NBUF = TEAMS == 1 ? ACC_BUFS : TEAMS, TW = EPI_WARPS / TEAMS;      // see k_umma_i8
    constexpr int NI2 = N_ISSUE;
    constexpr uint32_t RM = 2;                              // barrier pairs per ring slot (see RingCursor)
    static_assert(TEAMS == 1 || (!is_f4(BN) && NBUF * BN <= 512 && TW % 4 == 0), "teams: byte tiles whose buffers fit tensor memory");
    constexpr uint32_t TMEM_COLS2 = TEAMS == 1 ? Cfg<BN>::TMEM_COLS : (NBUF * BN <= 256 ? 256 : 512);
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Control *ctl = reinterpret_cast<Control *>(tiles + STAGES2 * STAGE2_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                // 0 = leader of the pair
    const int64_t pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    BNN_CLK_REC(0);
    const int64_t tiles_m = (p.M + 2 * BM - 1) / (2 * BM);  // 256-row tiles
    const int64_t tiles_n = (p.N + BN - 1) / BN;
    const int64_t ntiles = tiles_m * tiles_n;

    if (threadIdx.x == 0) {
        for (int s = 0; s < (int)RM * STAGES2; ++s) { mbar_init(smem_u32(&ctl->full[s]), 1); mbar_init(smem_u32(&ctl->empty[s]), 1); }
        for (int b = 0; b < NBUF; ++b) {
            mbar_init(smem_u32(&ctl->acc_full[b]), NI2);        // one multicast commit from each of the leader's MMA warps
            mbar_init(smem_u32(&ctl->acc_empty[b]), 2 * TW);    // the warps of the team that reads this buffer, in both CTAs
        }
        ctl->failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(TMEM_COLS2) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync_all();                                     // both CTAs' barriers exist before anyone signals them
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = ctl->tmem_base;

    {
        // Zero accumulators in this CTA's tensor memory (see tmem_zero32) and, on the 4-bit engine, unit block scales (byte
        // 0x7f) in its scale-factor columns; the leader's MMAs write / read the columns of both CTAs, so the pair
        // synchronises once more before the first one is issued
        if (warp >= 2 && warp < 6) {
            tmem_zero_all(tmem_base, warp, NBUF * BN);
            if (is_f4(BN)) {
                const uint32_t v = 0x7f7f7f7fu;
                asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1};"
                             ::"r"(tmem_base + SF_COL + ((uint32_t)(32 * (warp & 3)) << 16)), "r"(v) : "memory");
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        cluster_sync_all();
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    }

    if (warp == 0 || warp == Warps<BN>::PROD_WARP_B) {
        // ---------------- TMA producers (both CTAs): two threads, alternate K steps.  One thread needs ~500-700 clocks per K
        // step for its barrier poll, the byte count and two loads -- more than the 448-512 clocks in which the step is
        // multiplied -- so with one producer a tile ran at the producer's pace; each of two has twice the time.
        if (lane == 0) {
            // each producer thread takes every other K step of the pair's sequence, with both operands
            const uint32_t wp = (warp == 0) ? 0u : 1u;
            bool ok = true;
            RingCursor rc; rc.start(wp, STAGES2, RM);
            const uint32_t tn32 = (uint32_t)tiles_n;
            uint32_t it0 = 0;                            // K steps of this pair before the current tile
            // the weights of the first ring fill are requested before the wait for the preceding kernel (see k_umma_i8)
            const int npre = !p.b_static ? 0 : (p.k_iters < STAGES2 ? p.k_iters : STAGES2);
            {
                const int nb0f = (int)(((uint32_t)pair % tn32) * BN + rank * (BN / 2));
                for (int kit = (int)wp; kit < npre; kit += 2) {
                    if (rank == 0) mbar_expect_tx(smem_u32(&ctl->full[kit]), 2 * STAGE2_BYTES);
                    tma_load_2d_2sm(smem_u32(tiles + kit * STAGE2_BYTES + A_BYTES), &mapB, kit * BK, nb0f, smem_u32(&ctl->full[kit]) & PEER_MASK);
                }
            }
            bnn_pdl_wait();
            for (uint32_t t = (uint32_t)pair; t < (uint32_t)ntiles && ok; t += (uint32_t)npairs, it0 += (uint32_t)p.k_iters) {
                const bool first_tile = (t == (uint32_t)pair);
                const uint32_t tm = t / tn32;
                const int m0 = (int)(tm * (2 * BM) + rank * BM);
                const int nb0 = (int)((t - tm * tn32) * BN + rank * (BN / 2));
                int b0 = 0, y0 = 0;
                if (p.conv) {
                    // this CTA's 128 pixels of the pair's 256 (see k_umma_i8): first image and row, taps per K step
                    const int tm128 = 2 * (int)tm + (int)rank, tiles_per_img = p.H / p.TH;
                    b0 = (p.TB > 1) ? tm128 * p.TB : tm128 / tiles_per_img;
                    y0 = (p.TB > 1) ? 0 : (tm128 % tiles_per_img) * p.TH;
                }
                for (int kit = (int)((wp + it0) & 1u); kit < p.k_iters; kit += 2) {
                    const bool pre = first_tile && kit < npre;
                    if (kit < 8) BNN_TR(0, (t - (uint32_t)pair) / (uint32_t)npairs, kit);
                    if (rc.reuses(STAGES2) && !mbar_wait(ctl, p.wait_ns, smem_u32(&ctl->empty[rc.prev_bar(STAGES2, RM)]), rc.prev_parity(STAGES2))) { fail_pair(ctl, 11); ok = false; break; }
                    const uint32_t dst = smem_u32(tiles + rc.slot(STAGES2) * STAGE2_BYTES);
                    const uint32_t bar0 = smem_u32(&ctl->full[rc.b]) & PEER_MASK;
                    if (!pre && rank == 0) mbar_expect_tx(smem_u32(&ctl->full[rc.b]), 2 * STAGE2_BYTES);   // the bytes of both CTAs, both operands
                    if (p.conv) {
                        const int tap = kit / p.c_chunks, cc = kit - tap * p.c_chunks, ty = tap / 3;
                        tma_load_4d_2sm(dst, &mapA, cc * BK, tap - 3 * ty - 1, y0 + ty - 1, b0, bar0);
                    } else {
                        tma_load_2d_2sm(dst, &mapA, kit * BK, m0, bar0);
                    }
                    if (!pre) tma_load_2d_2sm(dst + A_BYTES, &mapB, kit * BK, nb0, bar0);
                    rc.advance(2, STAGES2, RM);
                }
            }
        }
    } else if (warp == 1 || warp == MMA_WARP_B) {
        // ---------------- MMA issuers: two warps of the leader CTA only (even / odd K steps), for both tensor cores.  A pair's
        // MMA costs the thread that issues it ~120 clocks, more than the tensor cores need for most shapes, so one thread
        // cannot keep them busy; two reach the pipe's rate in a loop of nothing else (measured: 112 clocks per 256 x 224
        // x 64 nibble MMA, 128 per 256 x 256 x 32 byte MMA, on one accumulator or two).
        if (lane == 0 && rank == 0) {
            const int w = (warp == 1) ? 0 : 1;
            // the host's descriptor carries M = 128 in bits [24,29); the pair multiplies M = 256
            const uint32_t idesc = is_f4(BN)
                ? ((1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | (1u << 23) | ((uint32_t)((2 * BM) >> 4) << 24))
                : ((p.idesc & ~(0x1fu << 24)) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24));
            const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
            const uint64_t adesc0 = smem_desc_sw128(smem_u32(tiles)), bdesc0 = smem_desc_sw128(smem_u32(tiles + A_BYTES));
            uint32_t it0 = 0, tc = 0;
            bool ok = true;
            for (int64_t t = pair; t < ntiles && ok; t += npairs, ++tc, it0 += (uint32_t)p.k_iters) {
                const uint32_t buf = tc % NBUF, use = tc / NBUF;
                if (use > 0 && !mbar_wait(ctl, p.wait_ns, smem_u32(&ctl->acc_empty[buf]), (use - 1) & 1)) { fail_pair(ctl, 14); ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                BNN_TR(1 + w, tc, 0);
                const uint32_t tmem_d = tmem_base + buf * BN;
                RingCursor rc; rc.start(it0 + w, STAGES2, RM);
                for (int kit = w; kit < p.k_iters; kit += NI2) {
                    const bool fine = (kit == 4 + w);         // instrumented builds: one steady-state K step per tile in detail
                    if (fine) BNN_TR(5 + w, tc, 0);
                    if (!mbar_wait(ctl, p.wait_ns, full0 + 8 * rc.b, rc.parity())) { fail_pair(ctl, 12); ok = false; break; }
                    if (fine) BNN_TR(5 + w, tc, 1);
                    const uint32_t s = rc.slot(STAGES2);
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    if (fine) BNN_TR(5 + w, tc, 2);
                    if (kit < 10) BNN_TR(1 + w, tc, 1 + kit);
                    const uint64_t adesc = adesc0 + (uint64_t)(s * (STAGE2_BYTES >> 4));
                    const uint64_t bdesc = bdesc0 + (uint64_t)(s * (STAGE2_BYTES >> 4));
                    const int nk = (kit == p.k_iters - 1) ? p.k_last : BK / 32;
#pragma unroll
                    for (int k = 0; k < BK / 32; ++k) {
                        if (k >= nk) break;
                        if (is_f4(BN)) umma_mxf4_2sm(tmem_d, adesc + 2 * k, bdesc + 2 * k, idesc, 1u, tmem_base + SF_COL);
                        else umma_i8_2sm(tmem_d, adesc + 2 * k, bdesc + 2 * k, idesc, 1u);
                        if (fine) BNN_TR(5 + w, tc, 3 + k);
                    }
                    umma_commit_2sm(empty0 + 8 * rc.b);
                    if (fine) BNN_TR(5 + w, tc, 7);
                    rc.advance(NI2, STAGES2, RM);
                }
                umma_commit_2sm(smem_u32(&ctl->acc_full[buf]));
                BNN_TR(1 + w, tc, 11);
            }
        }
    } else if (warp < 2 + EPI_WARPS) {
        // ---------------- epilogue (both CTAs): this CTA's 128 rows of the pair's tile
        bnn_pdl_wait();
        bnn_pdl_launch_next();
        const int q = warp & 3;
        const int team = (warp - 2) / TW;
        const int half = ((warp - 2) % TW) >> 2;
        const int et = (threadIdx.x - 64) % (32 * TW);
        bool ok = true;
        const uint32_t tn = (uint32_t)tiles_n, nt = (uint32_t)ntiles, np = (uint32_t)npairs;
        for (uint32_t tc = (uint32_t)team; ; tc += TEAMS) {
            const uint32_t t = (uint32_t)pair + tc * np;
            if (t >= nt) break;
            const uint32_t tm_i = t / tn;
            const int64_t m0 = (int64_t)tm_i * (2 * BM) + rank * BM, n0 = (int64_t)(t - tm_i * tn) * BN;
            const uint32_t t2 = t + TEAMS * np;
            const int64_t n0_next = (t2 < nt) ? (int64_t)(t2 % tn) * BN : -1;
            uint32_t buf;
            if constexpr (TEAMS == 1) {
                buf = tc & 1;
                epilogue_tile<BN>(ctl, p, tmem_base, buf, tc, m0, n0, n0_next, q, half, lane, et, ok, tc == 0, (tc / ACC_BUFS) & 1, buf ^ 1u);
            } else {
                buf = (uint32_t)team;
                const bool first = tc < (uint32_t)TEAMS, same = n0_next == n0;
                const uint32_t par = (tc / TEAMS) & 1u;
#define BNN_EPI_TEAM(K) epilogue_tile<BN, false, TW, K, false>(ctl, p, tmem_base, buf, tc, m0, n0, n0_next, q, half, lane, et, ok, first, par, buf, same)
                if (TEAMS > 3 && team == 3) BNN_EPI_TEAM((TEAMS > 3 ? 3 : 0));
                else if (TEAMS > 2 && team == 2) BNN_EPI_TEAM((TEAMS > 2 ? 2 : 0));
                else if (team == 1) BNN_EPI_TEAM(1);
                else BNN_EPI_TEAM(0);
#undef BNN_EPI_TEAM
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive_cta0(smem_u32(&ctl->acc_empty[buf]));
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    BNN_CLK_REC(1);
    cluster_sync_all();                                     // nobody leaves while the peer may still read its shared memory
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS2) : "memory");
    }
}

#include "bnn_umma_conv.cuh"

// ---------------------------------------------------------------------------------------------------------
// Packed signs -> one signed byte per value (+1 = 0x01, -1 = 0xff); bytes at or beyond K are 0.
// One thread per 32-bit word = 32 output bytes (two 128-bit stores).
// 32 bytes to a 32-byte aligned global address in one instruction (a whole sector per thread).
__device__ __forceinline__ void store_256(void *dst, const uint32_t (&v)[8]) {
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"l"(dst), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]) : "memory");
}
// Thread index -> (row, word of the row): 32-bit division whenever the launch has fewer than 2^32 threads' worth of words.
__device__ __forceinline__ void row_and_word(int64_t idx, int64_t wpr, int64_t total, int64_t &r, int64_t &w) {
    if (total <= 0xffffffffll) { const uint32_t rr = (uint32_t)idx / (uint32_t)wpr; r = rr; w = (uint32_t)idx - rr * (uint32_t)wpr; }
    else { r = idx / wpr; w = idx - r * wpr; }
}
__global__ void __launch_bounds__(256) k_expand_s8(const uint32_t *__restrict__ src, int64_t ld_w, int64_t rows, int64_t K,
                                                   int8_t *__restrict__ dst, int64_t ld8) {
    bnn_pdl_wait();
    bnn_pdl_launch_next();
    const int64_t wpr = ld8 >> 5;            // words per output row (ld8 is a multiple of 32)
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * wpr) return;
    int64_t r, w;
    row_and_word(idx, wpr, rows * wpr, r, w);
    const int64_t Kw = (K + 31) >> 5;
    uint32_t bits = 0u, valid = 0u;
    if (w < Kw) {
        bits = src[r * ld_w + w];
        valid = (w == Kw - 1 && (K & 31)) ? ((1u << (K & 31)) - 1u) : 0xffffffffu;
    }
    uint32_t b[8];
    if (valid == 0xffffffffu) {              // every word but a row's last one
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            const uint32_t t = (((bits >> (4 * g)) & 0xfu) * 0x00204081u) & 0x01010101u;      // 0/1 bytes
            b[g] = ~(t * 0xfeu);
        }
    } else {
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            const uint32_t t = (((bits >> (4 * g)) & 0xfu) * 0x00204081u) & 0x01010101u;
            const uint32_t v = (((valid >> (4 * g)) & 0xfu) * 0x00204081u) & 0x01010101u;
            b[g] = (~(t * 0xfeu)) & (v * 0xffu);
        }
    }
    int8_t *d = dst + r * ld8 + 32 * w;
    if ((reinterpret_cast<uintptr_t>(d) & 31u) == 0) {
        store_256(d, b);
    } else {
        reinterpret_cast<uint4 *>(d)[0] = make_uint4(b[0], b[1], b[2], b[3]);
        reinterpret_cast<uint4 *>(d)[1] = make_uint4(b[4], b[5], b[6], b[7]);
    }
}

// Packed signs -> one e2m1 nibble per value (+1.0 = 0x2, -1.0 = 0xa), two per byte, value k in byte k/2 (even k in
// the low nibble); nibbles at or beyond K are 0 (= +0.0).  One thread per two 32-bit words = 32 output bytes.
__device__ __forceinline__ void expand_word_f4(uint32_t bits, uint32_t valid, uint32_t *q) {
    if (valid == 0xffffffffu) {              // every word but a row's last one
#pragma unroll
        for (int g = 0; g < 4; ++g) q[g] = nibbles_of_byte((bits >> (8 * g)) & 0xffu);
    } else {
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            const uint32_t n = nibbles_of_byte((bits >> (8 * g)) & 0xffu);
            const uint32_t v = nibbles_of_byte((valid >> (8 * g)) & 0xffu);      // 0x2 where valid, 0xa where not
            q[g] = n & (((~v >> 3) & 0x11111111u) * 0xfu);                         // keep the nibbles whose valid bit is set
        }
    }
}
__global__ void __launch_bounds__(256) k_expand_f4(const uint32_t *__restrict__ src, int64_t ld_w, int64_t rows, int64_t K,
                                                   uint8_t *__restrict__ dst, int64_t ld4) {
    bnn_pdl_wait();
    bnn_pdl_launch_next();
    const int64_t ppr = ld4 >> 5;            // word pairs per output row (ld4 is a multiple of 128 bytes)
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * ppr) return;
    int64_t r, pw;
    row_and_word(idx, ppr, rows * ppr, r, pw);
    const int64_t Kw = (K + 31) >> 5, w = 2 * pw;
    const uint32_t last = (K & 31) ? ((1u << (K & 31)) - 1u) : 0xffffffffu;
    uint32_t bits[2] = {0u, 0u}, valid[2] = {0u, 0u};
    if (w + 1 < Kw) {                        // both words inside the row: one 64-bit load (rows are 16-byte aligned)
        const uint2 v = *reinterpret_cast<const uint2 *>(src + r * ld_w + w);
        bits[0] = v.x; bits[1] = v.y;
        valid[0] = 0xffffffffu; valid[1] = (w + 1 == Kw - 1) ? last : 0xffffffffu;
    } else if (w < Kw) {
        bits[0] = src[r * ld_w + w];
        valid[0] = (w == Kw - 1) ? last : 0xffffffffu;
    }
    uint32_t q[8];
    expand_word_f4(bits[0], valid[0], q);
    expand_word_f4(bits[1], valid[1], q + 4);
    uint8_t *d = dst + r * ld4 + 32 * pw;
    if ((reinterpret_cast<uintptr_t>(d) & 31u) == 0) {
        store_256(d, q);
    } else {
        reinterpret_cast<uint4 *>(d)[0] = make_uint4(q[0], q[1], q[2], q[3]);
        reinterpret_cast<uint4 *>(d)[1] = make_uint4(q[4], q[5], q[6], q[7]);
    }
}

// First convolution: the 3x3 neighbourhood of every pixel of an 8-bit NHWC image (9 * C_in <= 32 bytes, taps
// outside the image as zeros) written as one 32-byte row, byte (tap * C_in + c).  One thread per pixel.
// CIN > 0: the channel count as a compile-time constant (the packing below then stays in registers); 0: run-time Cin.
template <int CIN>
__global__ void __launch_bounds__(256) k_im2col_u8(const uint8_t *__restrict__ act, int64_t B, int H, int W, int Cin,
                                                   uint8_t *__restrict__ dst) {
    bnn_pdl_wait();
    bnn_pdl_launch_next();
    const int64_t pix = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (pix >= B * H * W) return;
    const int x = (int)(pix % W), y = (int)((pix / W) % H);
    const int64_t b = pix / ((int64_t)W * H);
    uint32_t w[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
    if (CIN > 0) {
#pragma unroll
        for (int tap = 0; tap < 9; ++tap) {
            const int yy = y + tap / 3 - 1, xx = x + tap % 3 - 1;
            if (yy < 0 || yy >= H || xx < 0 || xx >= W) continue;
            const uint8_t *px = act + ((b * H + yy) * W + xx) * CIN;
#pragma unroll
            for (int c = 0; c < CIN; ++c) {
                const int k = tap * CIN + c;
                w[k >> 2] |= (uint32_t)px[c] << (8 * (k & 3));
            }
        }
    } else {
        for (int tap = 0; tap < 9; ++tap) {
            const int yy = y + tap / 3 - 1, xx = x + tap % 3 - 1;
            if (yy < 0 || yy >= H || xx < 0 || xx >= W) continue;
            const uint8_t *px = act + ((b * H + yy) * W + xx) * Cin;
            for (int c = 0; c < Cin; ++c) {
                const int k = tap * Cin + c;
                w[k >> 2] |= (uint32_t)px[c] << (8 * (k & 3));
            }
        }
    }
    uint8_t *d = dst + pix * 32;
    if ((reinterpret_cast<uintptr_t>(d) & 31u) == 0) {
        store_256(d, w);
    } else {
        reinterpret_cast<uint4 *>(d)[0] = make_uint4(w[0], w[1], w[2], w[3]);
        reinterpret_cast<uint4 *>(d)[1] = make_uint4(w[4], w[5], w[6], w[7]);
    }
}

typedef CUresult (*encode_fn_t)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
std::mutex g_encode_mutex;
encode_fn_t g_encode = nullptr;

int get_encode(bnn_ctx *ctx, encode_fn_t *out) {
    std::lock_guard<std::mutex> lock(g_encode_mutex);
    if (!g_encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        BNN_CUDA_TRY(ctx, cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
        if (!fn || qres != cudaDriverEntryPointSuccess) return BNN_ERR_CUDA;
        g_encode = reinterpret_cast<encode_fn_t>(fn);
    }
    *out = g_encode;
    return BNN_OK;
}

// 2-D byte tensor rows x kbytes (row pitch ld bytes), box 128 bytes x box_rows, 128-byte swizzle, zero fill outside.
// box_k = 64: boxes of 64 bytes with the 64-byte swizzle (the halo-tile convolution's half-width K steps).
int make_map(bnn_ctx *ctx, CUtensorMap *map, const void *base, int64_t rows, int64_t kbytes, int64_t ld, int box_rows, int box_k = BK) {
    encode_fn_t enc;
    if (int st = get_encode(ctx, &enc)) return st;
    cuuint64_t dims[2] = {(cuuint64_t)kbytes, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld};
    cuuint32_t box[2] = {(cuuint32_t)box_k, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, box_k == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { ctx->last_cuda_error = (int)r; return BNN_ERR_CUDA; }
    return BNN_OK;
}

}  // namespace

template <int BN> static size_t umma_smem_bytes() { return (size_t)Cfg<BN>::STAGES * Cfg<BN>::STAGE_BYTES + sizeof(Control) + 1024; }
// Opt in to the large dynamic shared memory once per device.
static int umma_prepare(bnn_ctx *ctx) {
    static std::mutex attr_mutex;
    static bool attr_set[64] = {};
    std::lock_guard<std::mutex> lock(attr_mutex);
    if (ctx->device < 0 || ctx->device >= 64) return BNN_ERR_INVALID_ARG;
    if (!attr_set[ctx->device]) {
        BNN_CUDA_TRY(ctx, cudaFuncSetAttribute(k_umma_i8<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)umma_smem_bytes<256>()));
        BNN_CUDA_TRY(ctx, cudaFuncSetAttribute(k_umma_i8<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)umma_smem_bytes<128>()));
        BNN_CUDA_TRY(ctx, cudaFuncSetAttribute(k_umma_i8<192>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)umma_smem_bytes<192>()));
        BNN_CUDA_TRY(ctx, (cudaFuncSetAttribute(k_umma_i8<256, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)umma_smem_bytes<256>())));
        BNN_CUDA_TRY(ctx, (cudaFuncSetAttribute(k_umma_i8<128, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)umma_smem_bytes<128>())));
        attr_set[ctx->device] = true;
    }
    return BNN_OK;
}
// Tile width for N output columns: 128 when that leaves no (or less) idle MMA columns, or when 256-wide tiles would
// occupy less than half of the SMs (small batches).
static int umma_tile_n(int64_t N, int64_t M = 0, int sm_count = 0) {
    if (((N + 127) / 128) & 1) return 128;
    if (M > 0 && ((M + BM - 1) / BM) * ((N + 255) / 256) * 2 <= sm_count) return 128;
    return 256;
}
template <int BN> static size_t umma2_smem_bytes() { return (size_t)Cfg2<BN>::STAGES * Cfg2<BN>::STAGE_BYTES + sizeof(Control) + 1024; }
// Pairs of CTAs that can be resident at once for the two-SM kernel on this device (0 = cannot be used).
template <int BN, int TEAMS = 1>
static int umma2_max_pairs(bnn_ctx *ctx) {
    static std::mutex m;
    static int cached[64];
    static bool have[64] = {};
    std::lock_guard<std::mutex> lock(m);
    if (ctx->device < 0 || ctx->device >= 64) return 0;
    if (!have[ctx->device]) {
        int pairs = 0;
        if (cudaFuncSetAttribute(k_umma_i8_2sm<BN, TEAMS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)umma2_smem_bytes<BN>()) == cudaSuccess) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(2 * ctx->sm_count, 1, 1);
            cfg.blockDim = dim3(Warps<BN>::NTHREADS, 1, 1);
            cfg.dynamicSmemBytes = umma2_smem_bytes<BN>();
            cudaLaunchAttribute attr;
            attr.id = cudaLaunchAttributeClusterDimension;
            attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
            cfg.attrs = &attr; cfg.numAttrs = 1;
            if (cudaOccupancyMaxActiveClusters(&pairs, k_umma_i8_2sm<BN, TEAMS>, &cfg) != cudaSuccess) pairs = 0;
        }
        (void)cudaGetLastError();
        cached[ctx->device] = pairs;
        have[ctx->device] = true;
    }
    return cached[ctx->device];
}
// Epilogue teams (k_umma_i8<BN, TEAMS>) for byte-operand tiles whose K steps take less time than one tile's epilogue
// (~2500-3500 clocks): 4 x 64 clocks per K step at 128 columns, 4 x 128 at 256.
static bool umma_want_teams(const UmmaArgs &a, int bn) {
    if (!a.thr || a.conv || is_f4(bn) || (bn != 128 && bn != 256)) return false;
    return (int64_t)a.k_iters * 4 * (bn / 2) <= 4096;
}
static void note_kernel(bnn_ctx *ctx, const char *name, int bn, const char *operands, const char *extra = "") {
    snprintf(ctx->last_kernel, sizeof(ctx->last_kernel), "%s<%d> %s%s", name, bn, operands, extra);
}
static int umma_launch(bnn_ctx *ctx, const CUtensorMap &mapA, const CUtensorMap &mapB, const UmmaArgs &a, int bn) {
    if (int st = umma_prepare(ctx)) return st;
    note_kernel(ctx, "k_umma_i8", bn, is_f4(bn) ? "128 x bn tiles, tcgen05 kind::mxf4 on e2m1 nibbles" : "128 x bn tiles, tcgen05 kind::i8 on bytes");
    const int64_t tiles = ((a.M + BM - 1) / BM) * ((a.N + bn - 1) / bn);
    if (tiles >= (int64_t(1) << 31)) return BNN_ERR_INVALID_ARG;      // the kernels count tiles in 32 bits
    const int64_t grid = tiles < ctx->sm_count ? tiles : ctx->sm_count;
    const dim3 g((unsigned)grid);
    const bool teams = umma_want_teams(a, bn);
    if (teams) note_kernel(ctx, "k_umma_i8", bn, "128 x bn tiles, tcgen05 kind::i8 on bytes", bn == 128 ? ", 4 epilogue teams" : ", 2 epilogue teams");
    if (teams && bn == 256) BNN_CUDA_TRY(ctx, bnn_launch_dependent(k_umma_i8<256, 2>, g, dim3(Warps<256>::NTHREADS), umma_smem_bytes<256>(), ctx->stream, mapA, mapB, a));
    else if (teams) BNN_CUDA_TRY(ctx, bnn_launch_dependent(k_umma_i8<128, 4>, g, dim3(Warps<128>::NTHREADS), umma_smem_bytes<128>(), ctx->stream, mapA, mapB, a));
    else if (bn == 192) BNN_CUDA_TRY(ctx, bnn_launch_dependent(k_umma_i8<192>, g, dim3(Warps<192>::NTHREADS), umma_smem_bytes<192>(), ctx->stream, mapA, mapB, a));
    else if (bn == 256) BNN_CUDA_TRY(ctx, bnn_launch_dependent(k_umma_i8<256>, g, dim3(Warps<256>::NTHREADS), umma_smem_bytes<256>(), ctx->stream, mapA, mapB, a));
    else BNN_CUDA_TRY(ctx, bnn_launch_dependent(k_umma_i8<128>, g, dim3(Warps<128>::NTHREADS), umma_smem_bytes<128>(), ctx->stream, mapA, mapB, a));
    return bnn_check_launch(ctx);
}

size_t bnn_umma_operand_bytes(int64_t rows, int64_t K) {
    const int64_t ld8 = ((K + 127) / 128) * 128;
    return ((size_t)rows * ld8 + 255) & ~size_t(255);
}
int64_t bnn_umma_operand_ld(int64_t K) { return ((K + 127) / 128) * 128; }

int bnn_umma_expand(bnn_ctx *ctx, const uint32_t *src, int64_t ld_w, int64_t rows, int64_t K, int8_t *dst) {
    const int64_t ld8 = bnn_umma_operand_ld(K);
    const int64_t total = rows * (ld8 >> 5);
    if (total == 0) return BNN_OK;
    const int64_t blocks = (total + 255) / 256;
    if (blocks > 0x7fffffff) return BNN_ERR_INVALID_ARG;
    BNN_CUDA_TRY(ctx, bnn_launch_dependent(k_expand_s8, dim3((unsigned)blocks), dim3(256), 0, ctx->stream, src, ld_w, rows, K, dst, ld8));
    return bnn_check_launch(ctx);
}

// The 4-bit operand format: pitch and size of rows x K e2m1 nibbles.
int64_t bnn_umma_operand_ld_f4(int64_t K) { return ((K + 255) / 256) * 128; }
size_t bnn_umma_operand_bytes_f4(int64_t rows, int64_t K) { return ((size_t)rows * bnn_umma_operand_ld_f4(K) + 255) & ~size_t(255); }
int bnn_umma_expand_f4(bnn_ctx *ctx, const uint32_t *src, int64_t ld_w, int64_t rows, int64_t K, uint8_t *dst) {
    const int64_t ld4 = bnn_umma_operand_ld_f4(K);
    const int64_t total = rows * (ld4 >> 5);      // one thread per two words
    if (total == 0) return BNN_OK;
    const int64_t blocks = (total + 255) / 256;
    if (blocks > 0x7fffffff) return BNN_ERR_INVALID_ARG;
    BNN_CUDA_TRY(ctx, bnn_launch_dependent(k_expand_f4, dim3((unsigned)blocks), dim3(256), 0, ctx->stream, src, ld_w, rows, K, dst, ld4));
    return bnn_check_launch(ctx);
}

// Both operands as e2m1 nibbles (+-1 exactly; pitches in bytes): the same outputs as bnn_umma_gemm at twice the MMA
// rate and half the operand bytes.  Accumulation is float32, exact while K <= 2^24.  out4 (optional): the signs of
// the outputs as nibbles for a following layer, pitch ldo4 bytes.
int bnn_umma_gemm_f4(bnn_ctx *ctx, const uint8_t *A4, int64_t lda4, const uint8_t *B4, int64_t ldb4, int64_t M, int64_t N,
                     int64_t K, int32_t *C, int64_t ldc, const int32_t *thr, const uint32_t *flip, uint32_t *out, int64_t ldo,
                     uint8_t *out4, int64_t ldo4, int b_static) {
    if (M == 0 || N == 0) return BNN_OK;
    if ((lda4 & 15) || (ldb4 & 15) || !bnn_aligned16(A4) || !bnn_aligned16(B4)) return BNN_ERR_ALIGNMENT;
    if (M > 0x7fffffff || N > 0x7fffffff || K <= 0 || K > (1 << 24)) return BNN_ERR_INVALID_ARG;
    CUtensorMap mapA, mapB;
    const int64_t kb = (((K + 1) / 2 + 15) / 16) * 16;      // extent along K in bytes
    const bool pair_want = ctx->pair_mode == 2 || (ctx->pair_mode == 0 && (double)M * (double)N >= 6.0e6);
    // Pair kernel: 224- or 192-wide tiles.  A K step brings 128 + bn / 2 box rows into every CTA and the chip delivers
    // ~0.54 rows per clock and SM: 415 clocks for a 192-wide step whose MMAs take 384, but 444 clocks for a 224-wide one
    // whose MMAs take 448, so the wider tile is not held up by L2 and costs ~1.09 x the narrower one for 1.17 x the
    // columns (measured).  The kernel's time is the largest number of tiles one pair gets, times that cost.
    int bn2 = 192;
    {
        const int p224 = umma2_max_pairs<224>(ctx), p192 = umma2_max_pairs<192>(ctx);
        if (p224 > 0 && p192 > 0) {
            const int64_t tm2 = (M + 2 * BM - 1) / (2 * BM);
            const int64_t r224 = (tm2 * ((N + 223) / 224) + p224 - 1) / p224, r192 = (tm2 * ((N + 191) / 192) + p192 - 1) / p192;
            // (a B operand that does not stay in L2 between the row blocks makes the product wait for HBM instead:
            // 16384^3, 134 MB of B, measured 1.62 ms on 224-wide and 1.55 ms on 192-wide tiles)
            if (1.09 * (double)r224 <= (double)r192 && (double)N * (double)kb <= 6.4e7) bn2 = 224;
        } else if (p224 > 0) {
            bn2 = 224;
        }
    }
#ifdef BNN_F4_PAIR_TILE
    bn2 = BNN_F4_PAIR_TILE;
#endif
    const int pairs = (!(M >= 512 && pair_want) || ctx->drop_loads) ? 0 : (bn2 == 224 ? umma2_max_pairs<224>(ctx) : umma2_max_pairs<192>(ctx));
    if (int st = make_map(ctx, &mapA, A4, M, kb <= lda4 ? kb : lda4, lda4, BM)) return st;
    if (int st = make_map(ctx, &mapB, B4, N, kb <= ldb4 ? kb : ldb4, ldb4, pairs > 0 ? bn2 / 2 : 192)) return st;
    UmmaArgs a{};
    a.wait_ns = ctx->wait_limit_ns; a.drop_loads = ctx->drop_loads;
    a.M = M; a.N = N;
    a.k_iters = (int)((K + 2 * BK - 1) / (2 * BK));          // 256 values per 128-byte K step
    a.k_last = (int)((K - 2 * BK * (int64_t)(a.k_iters - 1) + 63) / 64);
    a.C = C; a.ldc = ldc; a.out = out; a.ldo = ldo; a.thr = thr; a.flip = flip;
    a.out8 = reinterpret_cast<int8_t *>(out4); a.ldo8 = ldo4; a.out_f4 = 1; a.b_static = b_static;
    if (pairs > 0) {
        if (int st = umma_prepare(ctx)) return st;
        const int64_t tiles2 = ((M + 2 * BM - 1) / (2 * BM)) * ((N + bn2 - 1) / bn2);
        if (tiles2 >= (int64_t(1) << 31)) return BNN_ERR_INVALID_ARG;
        const int64_t use = tiles2 < pairs ? tiles2 : pairs;
        note_kernel(ctx, "k_umma_i8_2sm", bn2, "CTA pairs, 256 x bn tiles, tcgen05 cta_group::2 kind::mxf4 on e2m1 nibbles");
        if (bn2 == 224)
            BNN_CUDA_TRY(ctx, bnn_launch_dependent(k_umma_i8_2sm<224>, dim3((unsigned)(2 * use)), dim3(Warps<224>::NTHREADS), umma2_smem_bytes<224>(),
                                                   ctx->stream, mapA, mapB, a));
        else
            BNN_CUDA_TRY(ctx, bnn_launch_dependent(k_umma_i8_2sm<192>, dim3((unsigned)(2 * use)), dim3(Warps<192>::NTHREADS), umma2_smem_bytes<192>(),
                                                   ctx->stream, mapA, mapB, a));
        return bnn_check_launch(ctx);
    }
    return umma_launch(ctx, mapA, mapB, a, 192);
}

// C / bits = A8 (M x K bytes, pitch lda8; unsigned if a_unsigned) times B8^T (N x K signed bytes, pitch ldb8).
int bnn_umma_gemm(bnn_ctx *ctx, const void *A8, int64_t lda8, bool a_unsigned, const int8_t *B8, int64_t ldb8, int64_t M,
                  int64_t N, int64_t K, int32_t *C, int64_t ldc, const int32_t *thr, const uint32_t *flip, uint32_t *out,
                  int64_t ldo, int8_t *out8, int64_t ldo8, int pool, int64_t H, int64_t W, int out_f4, int b_static) {
    if (M == 0 || N == 0) return BNN_OK;
    if (pool) {   // rows are pixels of H x W images in (b, y, x) order; 128-row tiles must hold whole 2x2 windows
        int TH, TB;
        if (!bnn_umma_conv_tiling(H, W, 1, &TH, &TB) || C || !out) return BNN_ERR_INVALID_ARG;
    }
    if ((lda8 & 15) || (ldb8 & 15) || !bnn_aligned16(A8) || !bnn_aligned16(B8)) return BNN_ERR_ALIGNMENT;
    if (M > 0x7fffffff || N > 0x7fffffff) return BNN_ERR_INVALID_ARG;
    if (K <= 0) return BNN_ERR_INVALID_ARG;      // callers route the empty product elsewhere
    if (K > (a_unsigned ? (1 << 22) : (1 << 30)) - 1) return BNN_ERR_INVALID_ARG;   // |accumulator| < 2^30 (thresholding subtracts)
    CUtensorMap mapA, mapB;
    const int bn = umma_tile_n(N, M, ctx->sm_count);
    const int64_t kb = ((K + 15) / 16) * 16;      // extent along K in bytes; beyond it TMA fills zeros
    // two-SM kernel: 256-wide tiles, at least two 256-row tiles, plain GEMM epilogues
    // (auto: where it measured faster -- from about 1500 x 4096 outputs on; below that the larger tiles leave SMs idle)
    const bool pair_shape = bn == 256 && M >= 512 && !pool;
    const bool pair_want = ctx->pair_mode == 2 || (ctx->pair_mode == 0 && (double)M * (double)N >= 6.0e6);
    const int pairs = (pair_shape && pair_want && !ctx->drop_loads) ? umma2_max_pairs<256>(ctx) : 0;
    if (int st = make_map(ctx, &mapA, A8, M, kb <= lda8 ? kb : lda8, lda8, BM)) return st;
    if (int st = make_map(ctx, &mapB, B8, N, kb <= ldb8 ? kb : ldb8, ldb8, pairs > 0 ? 128 : bn)) return st;
    UmmaArgs a{};
    a.wait_ns = ctx->wait_limit_ns; a.drop_loads = ctx->drop_loads;
    a.M = M; a.N = N;
    a.k_iters = (int)((K + BK - 1) / BK);
    a.k_last = (int)((K - BK * (int64_t)(a.k_iters - 1) + 31) / 32);
    a.idesc = (2u << 4) | ((a_unsigned ? 0u : 1u) << 7) | (1u << 10) | ((uint32_t)(BM >> 4) << 24);   // N field added by the kernel
    a.C = C; a.ldc = ldc; a.out = out; a.ldo = ldo; a.out8 = out8; a.ldo8 = ldo8; a.thr = thr; a.flip = flip;
    a.pool = pool; a.H = (int)H; a.W = (int)W; a.out_f4 = out_f4; a.b_static = b_static;
    if (pairs > 0) {
        const int64_t tiles2 = ((M + 2 * BM - 1) / (2 * BM)) * ((N + 255) / 256);
        if (tiles2 >= (int64_t(1) << 31)) return BNN_ERR_INVALID_ARG;
        const int64_t use = tiles2 < pairs ? tiles2 : pairs;
        if (umma_want_teams(a, 256) && umma2_max_pairs<256, 2>(ctx) >= pairs) {
            note_kernel(ctx, "k_umma_i8_2sm", 256, "CTA pairs, 256 x bn tiles, tcgen05 cta_group::2 kind::i8 on bytes", ", 2 epilogue teams");
            BNN_CUDA_TRY(ctx, (bnn_launch_dependent(k_umma_i8_2sm<256, 2>, dim3((unsigned)(2 * use)), dim3(Warps<256>::NTHREADS), umma2_smem_bytes<256>(),
                                                    ctx->stream, mapA, mapB, a)));
            return bnn_check_launch(ctx);
        }
        note_kernel(ctx, "k_umma_i8_2sm", 256, "CTA pairs, 256 x bn tiles, tcgen05 cta_group::2 kind::i8 on bytes");
        BNN_CUDA_TRY(ctx, bnn_launch_dependent(k_umma_i8_2sm<256>, dim3((unsigned)(2 * use)), dim3(Warps<256>::NTHREADS), umma2_smem_bytes<256>(),
                                               ctx->stream, mapA, mapB, a));
        return bnn_check_launch(ctx);
    }
    return umma_launch(ctx, mapA, mapB, a, bn);
}

namespace {
int make_map_nhwc(bnn_ctx *ctx, CUtensorMap *map, const void *base, int64_t B, int64_t H, int64_t W, int64_t C, int TW, int TH,
                  int TB) {
    encode_fn_t enc;
    if (int st = get_encode(ctx, &enc)) return st;
    cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)B};
    cuuint64_t strides[3] = {(cuuint64_t)C, (cuuint64_t)(W * C), (cuuint64_t)(H * W * C)};
    cuuint32_t box[4] = {(cuuint32_t)BK, (cuuint32_t)TW, (cuuint32_t)TH, (cuuint32_t)TB};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { ctx->last_cuda_error = (int)r; return BNN_ERR_CUDA; }
    return BNN_OK;
}
}  // namespace

int bnn_umma_im2col_u8(bnn_ctx *ctx, const uint8_t *act, int64_t B, int64_t H, int64_t W, int64_t C_in, uint8_t *dst) {
    const int64_t total = B * H * W;
    if (total == 0) return BNN_OK;
    const int64_t blocks = (total + 255) / 256;
    if (blocks > 0x7fffffff || 9 * C_in > 32) return BNN_ERR_INVALID_ARG;
    if (C_in == 3)
        BNN_CUDA_TRY(ctx, bnn_launch_dependent(k_im2col_u8<3>, dim3((unsigned)blocks), dim3(256), 0, ctx->stream, act, B, (int)H, (int)W, (int)C_in, dst));
    else if (C_in == 1)
        BNN_CUDA_TRY(ctx, bnn_launch_dependent(k_im2col_u8<1>, dim3((unsigned)blocks), dim3(256), 0, ctx->stream, act, B, (int)H, (int)W, (int)C_in, dst));
    else
        BNN_CUDA_TRY(ctx, bnn_launch_dependent(k_im2col_u8<0>, dim3((unsigned)blocks), dim3(256), 0, ctx->stream, act, B, (int)H, (int)W, (int)C_in, dst));
    return bnn_check_launch(ctx);
}

// How a 128-pixel tile is cut out of H x W images: TB images x TH rows x W columns.  Returns false if the
// geometry does not tile that way (the caller then uses the CUDA-core kernel).
bool bnn_umma_conv_tiling(int64_t H, int64_t W, int pool, int *TH, int *TB) {
    if (W < 1 || W > BM || (BM % W) != 0) return false;
    const int64_t rows = BM / W;                 // image rows per tile if one image were tall enough
    if (H >= rows) {
        if (H % rows) return false;
        *TH = (int)rows; *TB = 1;
    } else {
        if (rows % H) return false;
        *TH = (int)H; *TB = (int)(rows / H);
    }
    if (pool && ((*TH & 1) || (W & 1))) return false;
    return true;
}

// ---- halo-tile convolution kernel (bnn_umma_conv.cuh): geometry, shared-memory plan and launch
namespace {
constexpr size_t SMEM_OPT_IN = 227 * 1024;      // dynamic shared memory a CTA can opt in to on sm_100
// Activation map with the dimensions ordered (channel byte, column, image, row): a box of {128, W, TB, TH + 2} lands in
// shared memory as [row][image][column] rows of 128 bytes.  cb = bytes of channels per pixel.
int make_map_slab(bnn_ctx *ctx, CUtensorMap *map, const void *base, int64_t B, int64_t H, int64_t W, int64_t cb, int TH, int TB, int kb) {
    encode_fn_t enc;
    if (int st = get_encode(ctx, &enc)) return st;
    cuuint64_t dims[4] = {(cuuint64_t)cb, (cuuint64_t)W, (cuuint64_t)B, (cuuint64_t)H};
    cuuint64_t strides[3] = {(cuuint64_t)cb, (cuuint64_t)(H * W * cb), (cuuint64_t)(W * cb)};
    cuuint32_t box[4] = {(cuuint32_t)kb, (cuuint32_t)W, (cuuint32_t)TB, (cuuint32_t)(TH + 2)};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, kb == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { ctx->last_cuda_error = (int)r; return BNN_ERR_CUDA; }
    return BNN_OK;
}
// Launch with programmatic stream serialization and, for the pair form, clusters of two CTAs.
template <typename... KArgs, typename... Args>
cudaError_t launch_conv_kernel(void (*kernel)(KArgs...), bool pair, dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args &&...args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = pair ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
// Per instantiation and device: opt in to the large shared memory once; for the pair form also ask how many clusters of
// two can be resident at once (0 = the pair form cannot be used).
template <int BN, bool F4, bool PAIR>
int conv_kernel_prepare(bnn_ctx *ctx, int *max_pairs) {
    static std::mutex m;
    static bool done[64] = {};
    static int pairs[64] = {};
    std::lock_guard<std::mutex> lock(m);
    if (ctx->device < 0 || ctx->device >= 64) return BNN_ERR_INVALID_ARG;
    if (!done[ctx->device]) {
        BNN_CUDA_TRY(ctx, cudaFuncSetAttribute(k_umma_conv<BN, F4, PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_OPT_IN));
        if (PAIR) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(2 * ctx->sm_count, 1, 1);
            cfg.blockDim = dim3(ConvCfg<BN, F4, PAIR>::NTHREADS, 1, 1);
            cfg.dynamicSmemBytes = SMEM_OPT_IN;
            cudaLaunchAttribute attr;
            attr.id = cudaLaunchAttributeClusterDimension;
            attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
            cfg.attrs = &attr; cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, k_umma_conv<BN, F4, PAIR>, &cfg) != cudaSuccess) n = 0;
            (void)cudaGetLastError();
            pairs[ctx->device] = n;
        }
        done[ctx->device] = true;
    }
    if (max_pairs) *max_pairs = pairs[ctx->device];
    return BNN_OK;
}
template <int BN, bool F4, bool PAIR>
int conv_halo_launch_t(bnn_ctx *ctx, const CUtensorMap &mapA, const CUtensorMap &mapB, const UmmaArgs &a, unsigned grid, size_t smem) {
    BNN_CUDA_TRY(ctx, launch_conv_kernel(k_umma_conv<BN, F4, PAIR>, PAIR, dim3(grid), dim3(ConvCfg<BN, F4, PAIR>::NTHREADS), smem, ctx->stream, mapA, mapB, a));
    return bnn_check_launch(ctx);
}
}  // namespace

// Whether the halo-tile kernel takes this layer: slabs of whole 1024-byte swizzle periods per image row of the tile.
static bool conv_halo_ok(const bnn_ctx *ctx, int64_t W, int TH, int TB, int kb = BK) {
    if (ctx->conv_form == 1 || ctx->drop_loads) return false;
    return ((TB * W) % 8) == 0 && W <= 256 && TB <= 256 && TH + 2 <= 256 && (size_t)(TH + 2) * TB * W * kb <= 48 * 1024;
}

// act: [B][H][W][cb] bytes (cb = C_in bytes, or C_in / 2 for nibbles; a multiple of 128), Wt: [C_out][9 * cb].  `a` arrives
// with the outputs, thresholds, pooling and tile geometry filled in.
// w_pitch: bytes between the filters' rows of Wt.  cb = 64 (128 channels as nibbles): K steps of 64 bytes.
static int conv_halo_launch(bnn_ctx *ctx, bool f4, const void *act, const void *Wt, int64_t w_pitch, int64_t B, int64_t H, int64_t W,
                            int64_t cb, int64_t C_out, int TH, int TB, UmmaArgs a, int b_static) {
    const int kb = cb == 64 ? 64 : BK;
    const int c_chunks = (int)(cb / kb);
    const size_t a_stage = (size_t)(TH + 2) * TB * W * kb;
    const size_t avail = SMEM_OPT_IN - 1024 - sizeof(Control);
    // 1. CTA pairs with the tile's filters resident, half of them in each CTA: 256 filters per tile on bytes, 128 on nibbles
    //    (two accumulator buffers and the scale columns must fit the 512 columns of tensor memory).
    bool pair = false, resident = false;
    int bn = 128, nb = 0, max_pairs = 0;
    if (ctx->pair_mode != 1 && a.M > BM) {
        bn = f4 ? 128 : (C_out > 128 ? 256 : 128);
        nb = 9 * c_chunks;
        int st = BNN_OK;
        if (f4) st = conv_kernel_prepare<128, true, true>(ctx, &max_pairs);
        else if (bn == 256) st = conv_kernel_prepare<256, false, true>(ctx, &max_pairs);
        else st = conv_kernel_prepare<128, false, true>(ctx, &max_pairs);
        if (st) return st;
        const int64_t tn = (C_out + bn - 1) / bn;
        pair = resident = max_pairs > 0 && nb <= B_STAGES_MAX && (size_t)nb * (bn / 2) * kb + 2 * a_stage <= avail && tn <= max_pairs;
    }
    // 2. otherwise one CTA per tile: resident weights where 128 filters fit, else streamed through a ring
    if (!pair) {
        bn = 128;
        resident = c_chunks == 1 && 9 * (size_t)128 * kb + 2 * a_stage <= avail && (C_out + 127) / 128 <= ctx->sm_count;
        if (!resident && C_out > 128) bn = f4 ? 192 : 256;
        nb = resident ? 9 : 4;
        int st = BNN_OK;
        if (f4) st = bn == 128 ? conv_kernel_prepare<128, true, false>(ctx, nullptr) : conv_kernel_prepare<192, true, false>(ctx, nullptr);
        else st = bn == 128 ? conv_kernel_prepare<128, false, false>(ctx, nullptr) : conv_kernel_prepare<256, false, false>(ctx, nullptr);
        if (st) return st;
    }
    const size_t b_stage = (size_t)(pair ? bn / 2 : bn) * kb, b_bytes = (size_t)nb * b_stage;
    int na = (int)((avail - b_bytes) / a_stage);
    na = na > 4 ? 4 : na;
    if (na < 2) return BNN_ERR_INVALID_ARG;
    CUtensorMap mapA, mapB;
    if (int st = make_map_slab(ctx, &mapA, act, B, H, W, cb, TH, TB, kb)) return st;
    if (int st = make_map(ctx, &mapB, Wt, C_out, 9 * cb, w_pitch, (int)(b_stage / kb), kb)) return st;
    a.conv = 1; a.H = (int)H; a.W = (int)W; a.TH = TH; a.TB = TB; a.c_chunks = c_chunks;
    a.k_iters = 9 * c_chunks; a.k_last = kb / 32; a.kbytes = kb;
    a.a_stage_bytes = (int)a_stage; a.n_a_stages = na; a.n_b_stages = nb; a.b_resident = resident ? 1 : 0;
    a.dy_bytes = (int)(TB * W * kb); a.tap_bytes = (int)cb; a.perm = TB > 1 ? 1 : 0; a.b_static = b_static;
    const int64_t tn = (C_out + bn - 1) / bn;
    const int64_t tile_m = pair ? 2 * BM : BM, tiles = ((a.M + tile_m - 1) / tile_m) * tn;
    if (tiles >= (int64_t(1) << 31)) return BNN_ERR_INVALID_ARG;
    const int64_t units_max = pair ? max_pairs : ctx->sm_count;
    int64_t units = tiles < units_max ? tiles : units_max;
    if (resident && tiles > units) units = (units_max / tn) * tn;       // a multiple of the filter blocks: one block per CTA (pair)
    const unsigned grid = (unsigned)(pair ? 2 * units : units);
    const size_t smem = (size_t)na * a_stage + b_bytes + sizeof(Control) + 1024;
    note_kernel(ctx, "k_umma_conv", bn, f4 ? "halo tiles, kind::mxf4 on e2m1 nibbles" : "halo tiles, kind::i8 on bytes",
                pair ? (resident ? ", CTA pairs, resident weights" : ", CTA pairs") : (resident ? ", resident weights" : ", streamed weights"));
    if (pair) {
        if (f4) return conv_halo_launch_t<128, true, true>(ctx, mapA, mapB, a, grid, smem);
        return bn == 256 ? conv_halo_launch_t<256, false, true>(ctx, mapA, mapB, a, grid, smem)
                         : conv_halo_launch_t<128, false, true>(ctx, mapA, mapB, a, grid, smem);
    }
    if (f4) return bn == 128 ? conv_halo_launch_t<128, true, false>(ctx, mapA, mapB, a, grid, smem)
                             : conv_halo_launch_t<192, true, false>(ctx, mapA, mapB, a, grid, smem);
    return bn == 128 ? conv_halo_launch_t<128, false, false>(ctx, mapA, mapB, a, grid, smem)
                     : conv_halo_launch_t<256, false, false>(ctx, mapA, mapB, a, grid, smem);
}

// 3x3 / pad 1 convolution on the tensor engine.  act8: [B][H][W][C_in] +-1 bytes (C_in % 128 == 0);
// W8: [C_out][9 * C_in] +-1 bytes.  Outputs as bnn_binary_conv2d (sums only without pooling).
int bnn_umma_conv(bnn_ctx *ctx, const int8_t *act8, const int8_t *W8, int64_t B, int64_t H, int64_t W, int64_t C_in,
                  int64_t C_out, int pool, const int32_t *thr, const uint32_t *flip, uint32_t *out_bits, int32_t *out_sums,
                  int8_t *out8, int64_t ldo8, int out_f4, int b_static) {
    int TH, TB;
    if (!bnn_umma_conv_tiling(H, W, pool, &TH, &TB) || (C_in % BK) != 0 || (pool && (out_sums || !out_bits))) return BNN_ERR_INVALID_ARG;
    if (conv_halo_ok(ctx, W, TH, TB)) {
        UmmaArgs h{};
        h.wait_ns = ctx->wait_limit_ns;
        h.M = B * H * W; h.N = C_out;
        h.idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BM >> 4) << 24);
        h.C = out_sums; h.ldc = C_out; h.out = out_bits; h.ldo = (C_out + 31) / 32; h.thr = thr; h.flip = flip;
        h.out8 = out8; h.ldo8 = ldo8; h.out_f4 = out_f4; h.pool = pool;
        return conv_halo_launch(ctx, false, act8, W8, bnn_umma_operand_ld(9 * C_in), B, H, W, C_in, C_out, TH, TB, h, b_static);
    }
    CUtensorMap mapA, mapB;
    const int bn = umma_tile_n(C_out);
    // CTA pairs (each CTA its own 128 pixels and half of the tile's filters) from 6 M outputs on, as for plain products
    const bool pair_want = ctx->pair_mode == 2 || (ctx->pair_mode == 0 && (double)(B * H * W) * (double)C_out >= 6.0e6);
    const int pairs = (!(B * H * W >= 512 && pair_want) || ctx->drop_loads) ? 0 : (bn == 256 ? umma2_max_pairs<256>(ctx) : umma2_max_pairs<128>(ctx));
    if (pairs > 0) { if (int st = umma_prepare(ctx)) return st; }
    if (int st = make_map_nhwc(ctx, &mapA, act8, B, H, W, C_in, (int)W, TH, TB)) return st;
    if (int st = make_map(ctx, &mapB, W8, C_out, 9 * C_in, 9 * C_in, pairs > 0 ? bn / 2 : bn)) return st;
    UmmaArgs a{};
    a.wait_ns = ctx->wait_limit_ns; a.drop_loads = ctx->drop_loads;
    a.M = B * H * W; a.N = C_out;
    a.k_iters = (int)(9 * (C_in / BK));
    a.k_last = BK / 32;
    a.idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BM >> 4) << 24);
    a.C = out_sums; a.ldc = C_out; a.out = out_bits; a.ldo = (C_out + 31) / 32; a.thr = thr; a.flip = flip;
    a.out8 = out8; a.ldo8 = ldo8; a.out_f4 = out_f4;
    a.conv = 1; a.H = (int)H; a.W = (int)W; a.TH = TH; a.TB = TB; a.c_chunks = (int)(C_in / BK); a.pool = pool;
    if (pairs > 0) {
        const int64_t tiles2 = ((a.M + 2 * BM - 1) / (2 * BM)) * ((C_out + bn - 1) / bn);
        if (tiles2 >= (int64_t(1) << 31)) return BNN_ERR_INVALID_ARG;
        const dim3 grid((unsigned)(2 * (tiles2 < pairs ? tiles2 : pairs)));
        if (bn == 256) BNN_CUDA_TRY(ctx, bnn_launch_dependent(k_umma_i8_2sm<256>, grid, dim3(Warps<256>::NTHREADS), umma2_smem_bytes<256>(), ctx->stream, mapA, mapB, a));
        else BNN_CUDA_TRY(ctx, bnn_launch_dependent(k_umma_i8_2sm<128>, grid, dim3(Warps<128>::NTHREADS), umma2_smem_bytes<128>(), ctx->stream, mapA, mapB, a));
        return bnn_check_launch(ctx);
    }
    return umma_launch(ctx, mapA, mapB, a, bn);
}

// The same convolution on 4-bit operands: act4 [B][H][W][C_in / 2] and W4 [C_out][9 * C_in / 2] bytes of e2m1 nibbles
// (C_in % 256 == 0, so that a K step is one tap and 256 channels = 128 bytes per pixel); pixels outside the image arrive
// as zero nibbles (+0.0).  Outputs: packed signs and / or nibbles for the next layer (out4, pitch ldo4 bytes per pixel),
// or the int32 sums (not with pooling).
// Whether the 4-bit engine takes a layer with C_in input maps: whole 128-byte channel slices (256 maps) in either form
// of the kernel, or exactly 128 maps (64 bytes per pixel) as half-width K steps of the halo-tile kernel.
bool bnn_umma_conv_f4_takes(const bnn_ctx *ctx, int64_t H, int64_t W, int pool, int64_t C_in) {
    if (C_in > 0 && (C_in % (2 * BK)) == 0) return true;
    int TH, TB;
    return C_in == BK && bnn_umma_conv_tiling(H, W, pool, &TH, &TB) && conv_halo_ok(ctx, W, TH, TB, 64);
}

int bnn_umma_conv_f4(bnn_ctx *ctx, const uint8_t *act4, const uint8_t *W4, int64_t B, int64_t H, int64_t W, int64_t C_in,
                     int64_t C_out, int pool, const int32_t *thr, const uint32_t *flip, uint32_t *out_bits, uint8_t *out4,
                     int64_t ldo4, int32_t *out_sums, int b_static) {
    int TH, TB;
    if (!bnn_umma_conv_tiling(H, W, pool, &TH, &TB) || !bnn_umma_conv_f4_takes(ctx, H, W, pool, C_in) || (pool && (out_sums || !out_bits)) ||
        (!out_bits && !out4 && !out_sums) || ((out_bits || out4) && !thr))
        return BNN_ERR_INVALID_ARG;
    if (!bnn_aligned16(act4) || !bnn_aligned16(W4)) return BNN_ERR_ALIGNMENT;
    if (conv_halo_ok(ctx, W, TH, TB, C_in == BK ? 64 : BK)) {
        UmmaArgs h{};
        h.wait_ns = ctx->wait_limit_ns;
        h.M = B * H * W; h.N = C_out;
        h.C = out_sums; h.ldc = C_out; h.out = out_bits; h.ldo = (C_out + 31) / 32; h.thr = thr; h.flip = flip;
        h.out8 = reinterpret_cast<int8_t *>(out4); h.ldo8 = ldo4; h.out_f4 = 1; h.pool = pool;
        return conv_halo_launch(ctx, true, act4, W4, bnn_umma_operand_ld_f4(9 * C_in), B, H, W, C_in / 2, C_out, TH, TB, h, b_static);
    }
    CUtensorMap mapA, mapB;
    // CTA pairs (each CTA its own 128 pixels and half of the tile's filters) cut the operand bytes per CTA by 30 %, but
    // measured slower on the ConvNet's layers (0.162 against 0.158 ms per batch of 256): on request only
    const int pairs = (ctx->pair_mode == 2 && B * H * W >= 512 && !ctx->drop_loads) ? umma2_max_pairs<192>(ctx) : 0;
    if (pairs > 0) { if (int st = umma_prepare(ctx)) return st; }
    if (int st = make_map_nhwc(ctx, &mapA, act4, B, H, W, C_in / 2, (int)W, TH, TB)) return st;
    if (int st = make_map(ctx, &mapB, W4, C_out, 9 * C_in / 2, 9 * C_in / 2, pairs > 0 ? 96 : 192)) return st;
    UmmaArgs a{};
    a.wait_ns = ctx->wait_limit_ns; a.drop_loads = ctx->drop_loads;
    a.M = B * H * W; a.N = C_out;
    a.c_chunks = (int)(C_in / (2 * BK));
    a.k_iters = 9 * a.c_chunks;
    a.k_last = BK / 32;
    a.C = out_sums; a.ldc = C_out; a.out = out_bits; a.ldo = (C_out + 31) / 32; a.thr = thr; a.flip = flip;
    a.out8 = reinterpret_cast<int8_t *>(out4); a.ldo8 = ldo4; a.out_f4 = 1;
    a.conv = 1; a.H = (int)H; a.W = (int)W; a.TH = TH; a.TB = TB; a.pool = pool;
    if (pairs > 0) {
        const int64_t tiles2 = ((a.M + 2 * BM - 1) / (2 * BM)) * ((C_out + 191) / 192);
        if (tiles2 >= (int64_t(1) << 31)) return BNN_ERR_INVALID_ARG;
        const int64_t use = tiles2 < pairs ? tiles2 : pairs;
        BNN_CUDA_TRY(ctx, bnn_launch_dependent(k_umma_i8_2sm<192>, dim3((unsigned)(2 * use)), dim3(Warps<192>::NTHREADS), umma2_smem_bytes<192>(),
                                               ctx->stream, mapA, mapB, a));
        return bnn_check_launch(ctx);
    }
    return umma_launch(ctx, mapA, mapB, a, 192);
}

extern "C" int64_t bnn_expanded_ld(int64_t K) { return K > 0 ? bnn_umma_operand_ld(K) : 0; }
extern "C" size_t bnn_expanded_bytes(int64_t rows, int64_t K) { return (rows > 0 && K > 0) ? bnn_umma_operand_bytes(rows, K) : 0; }
extern "C" int bnn_expand_signs(bnn_ctx *ctx, const uint32_t *src, int64_t ld_w, int64_t rows, int64_t K, int8_t *dst) {
    if (rows < 0 || K < 0) return BNN_ERR_INVALID_ARG;
    if (rows > 0 && K > 0) {   // the layout first: its errors need no context to be found
        if (!src || !dst) return BNN_ERR_INVALID_ARG;
        if (int st = bnn_check_packed(src, ld_w, K, rows)) return st;      // the kernels read the rows with 64- and 128-bit loads
        if (!bnn_aligned16(dst)) return BNN_ERR_ALIGNMENT;
    }
    if (!ctx) return BNN_ERR_INVALID_ARG;
    if (rows == 0 || K == 0) return BNN_OK;
    bnn_device_guard guard(ctx);
    if (!guard.ok) return BNN_ERR_CUDA;
    return bnn_umma_expand(ctx, src, ld_w, rows, K, dst);
}

extern "C" int64_t bnn_expanded_ld_f4(int64_t K) { return K > 0 ? bnn_umma_operand_ld_f4(K) : 0; }
extern "C" size_t bnn_expanded_bytes_f4(int64_t rows, int64_t K) { return (rows > 0 && K > 0) ? bnn_umma_operand_bytes_f4(rows, K) : 0; }
extern "C" int bnn_expand_signs_f4(bnn_ctx *ctx, const uint32_t *src, int64_t ld_w, int64_t rows, int64_t K, uint8_t *dst) {
    if (rows < 0 || K < 0) return BNN_ERR_INVALID_ARG;
    if (rows > 0 && K > 0) {
        if (!src || !dst) return BNN_ERR_INVALID_ARG;
        if (int st = bnn_check_packed(src, ld_w, K, rows)) return st;
        if (!bnn_aligned16(dst)) return BNN_ERR_ALIGNMENT;
    }
    if (!ctx) return BNN_ERR_INVALID_ARG;
    if (rows == 0 || K == 0) return BNN_OK;
    bnn_device_guard guard(ctx);
    if (!guard.ok) return BNN_ERR_CUDA;
    return bnn_umma_expand_f4(ctx, src, ld_w, rows, K, dst);
}

// Reads (and clears) the error word the tensor-core kernel sets when one of its bounded waits gives up.
// Synchronises the context's stream.
#ifdef BNN_TRACE
extern "C" BNN_API int bnn_trace_read(long long *host, int clear) {
    if (cudaMemcpyFromSymbol(host, g_trace, sizeof(long long) * 8 * 16 * 16) != cudaSuccess) return BNN_ERR_CUDA;
    if (clear) { static long long z[8 * 16 * 16]; if (cudaMemcpyToSymbol(g_trace, z, sizeof(z)) != cudaSuccess) return BNN_ERR_CUDA; }
    return BNN_OK;
}
#endif

// Host-side view of the ring arithmetic the kernels use (RingCursor), for tests without a GPU.
extern "C" int bnn_debug_ring_position(uint32_t stage, uint32_t slots, uint32_t step, uint32_t *slot, uint32_t *barrier,
                                       uint32_t *parity, int32_t *reuses, uint32_t *prev_barrier, uint32_t *prev_parity,
                                       uint32_t *next_barrier, uint32_t *next_parity) {
    if (slots == 0 || step == 0 || step > 2 * slots || !slot || !barrier || !parity || !reuses || !prev_barrier || !prev_parity ||
        !next_barrier || !next_parity)
        return BNN_ERR_INVALID_ARG;
    RingCursor rc;
    rc.start(stage, slots);
    *slot = rc.slot(slots); *barrier = rc.b; *parity = rc.parity();
    *reuses = rc.reuses(slots) ? 1 : 0;
    *prev_barrier = rc.reuses(slots) ? rc.prev_bar(slots) : 0u;
    *prev_parity = rc.reuses(slots) ? rc.prev_parity(slots) : 0u;
    rc.advance(step, slots);
    *next_barrier = rc.b; *next_parity = rc.parity();
    return BNN_OK;
}

extern "C" int bnn_last_tensor_kernel_clock(bnn_ctx *ctx, double *sm_mhz, double *microseconds) {
    if (!ctx || !sm_mhz || !microseconds) return BNN_ERR_INVALID_ARG;
    bnn_device_guard guard(ctx);
    if (!guard.ok) return BNN_ERR_CUDA;
    BNN_CUDA_TRY(ctx, cudaStreamSynchronize(ctx->stream));
    long long c[4] = {0, 0, 0, 0};
    BNN_CUDA_TRY(ctx, cudaMemcpyFromSymbol(c, g_umma_clock, sizeof(c)));
    const double ns = (double)(c[3] - c[1]);
    *microseconds = ns / 1e3;
    *sm_mhz = ns > 0 ? (double)(c[2] - c[0]) / ns * 1e3 : 0.0;
    return BNN_OK;
}

extern "C" int bnn_device_status(bnn_ctx *ctx) {
    if (!ctx) return BNN_ERR_INVALID_ARG;
    bnn_device_guard guard(ctx);
    if (!guard.ok) return BNN_ERR_CUDA;
    BNN_CUDA_TRY(ctx, cudaStreamSynchronize(ctx->stream));
    int code = 0;
    BNN_CUDA_TRY(ctx, cudaMemcpyFromSymbol(&code, g_umma_error, sizeof(int)));
    if (code != 0) {
        const int zero = 0;
        BNN_CUDA_TRY(ctx, cudaMemcpyToSymbol(g_umma_error, &zero, sizeof(int)));
        return BNN_ERR_DEVICE_STATUS;
    }
    return BNN_OK;
}
