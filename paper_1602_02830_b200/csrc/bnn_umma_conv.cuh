// Halo-tile form of the 3x3 / pad-1 binary convolution on the tensor cores (Section 3.3: every filter applied to the
// map as XNOR-popcount MACs, evaluated here as exact +-1 products).  Included by bnn_umma.cu, whose barrier, TMA,
// tcgen05 and epilogue helpers it uses.
//
// The implicit GEMM of a 128-pixel tile runs over nine taps.  Loading one 128-pixel operand box per tap (as the plain
// kernel k_umma_i8 does in its convolution mode) brings every input pixel into shared memory nine times, and what
// limits those layers is the rate at which L2 delivers box rows, not the tensor pipe.  Here a tile of TB images x TH
// rows x W columns loads, per horizontal tap dx and 128-byte channel slice, ONE slab of (TH + 2) x TB x W pixels whose
// column coordinate is shifted by dx (columns outside the image arrive as zeros from TMA, as do rows above and below
// it).  The slab is laid out [row][image][column], so the operand of vertical tap dy is the same slab read from an
// offset of (dy + 1) rows = (dy + 1) * TB * W * 128 bytes: a multiple of 1024 bytes (TB * W is a multiple of 8), i.e. a
// whole number of 128-byte-swizzle periods, so the shifted view is an ordinary K-major operand descriptor.  Three slabs
// instead of nine boxes per channel slice: the input traffic from L2 drops to (TH + 2) / (3 TH) of the plain form.
//
// The weights of the tile's BN filters are streamed through a ring of BN x 128-byte stages, one per (tap, slice) -- or,
// when all of them fit beside the slabs (BN = 128 and 128 bytes of channels per pixel: 144 KB), loaded ONCE per CTA and
// kept: the grid is then a multiple of the number of filter blocks, so every tile of a CTA uses the same filters.
//
// PAIR: two CTAs of a cluster work on one 256-pixel x BN tile with tcgen05.mma cta_group::2.  Each CTA loads the slabs
// of its own 128 pixels and keeps HALF of the tile's filters; the leader's thread issues for both tensor cores.  An MMA
// of M = 128 and N = 128 reads 8 KB of operands from its CTA's shared memory in its 64 clocks -- all the bandwidth shared
// memory has -- so in the single-CTA form every other shared-memory access (barrier polls, the epilogue's thresholds, the
// slabs being written) waits for gaps between MMAs and the issuing thread, which polls barriers in shared memory, falls
// behind: measured 40 % of the tensor pipe's rate.  The pair form reads 4 + 2 KB (BN = 128) or 4 + 4 KB per 128 clocks
// (BN = 256) per CTA.
//
// Roles: warp 0 producer, warp 1 and the last warp issue the MMAs (alternate slabs), the warps between run the epilogue (threshold, Sign, optional 2x2 pooling as OR of the sign bits, packed words and the next
// layer's operand format).  K step kit = (slice * 3 + dxi) * 3 + dyi multiplies the slab of (slice, dxi), viewed at row
// offset dyi, by the weights of tap 3 * dyi + dxi.
#pragma once

template <bool PAIR> __device__ __forceinline__ void conv_fail(Control *ctl, int code) {
    if (PAIR) fail_pair(ctl, code); else fail(ctl, code);
}

template <int BN, bool F4, bool PAIR> struct ConvCfg {
    static constexpr int EPI_WARPS = (BN == 192) ? 8 : 16;
    static constexpr int MMA_WARP_B = 2 + EPI_WARPS;                    // the second MMA-issuing warp (the first is warp 1)
    static constexpr int NTHREADS = 64 + 32 * EPI_WARPS + 32;
    static constexpr uint32_t B_ROWS = PAIR ? BN / 2 : BN;              // a CTA of a pair keeps half of the tile's filters
    static constexpr uint32_t TMEM_COLS = F4 ? 512 : (2 * BN <= 256 ? 256 : 512);
};

template <int BN, bool F4, bool PAIR>
__global__ void __launch_bounds__((ConvCfg<BN, F4, PAIR>::NTHREADS), 1)
k_umma_conv(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, const UmmaArgs p) {
    using C = ConvCfg<BN, F4, PAIR>;
    constexpr int EPI_WARPS = C::EPI_WARPS, MMA_WARP_B = C::MMA_WARP_B;
    constexpr uint32_t TMEM_COLS = C::TMEM_COLS;
    // K step: 128 bytes of channels per pixel (128-byte swizzle), or 64 bytes (64-byte swizzle: 128 maps as nibbles, two
    // MMAs per step); the vertical-tap offset TB * W * KB is a whole number of swizzle periods (8 rows) in both
    const int KB = p.kbytes;
    const uint32_t B_STAGE = C::B_ROWS * (uint32_t)KB;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *slabs = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t A_STAGE = (uint32_t)p.a_stage_bytes;
    const int NA = p.n_a_stages, NB = p.n_b_stages;
    uint8_t *wts = slabs + (size_t)NA * A_STAGE;
    Control *ctl = reinterpret_cast<Control *>(wts + (size_t)NB * B_STAGE);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;                 // 0 = the pair's leader
    const uint32_t unit = PAIR ? (blockIdx.x >> 1) : blockIdx.x;         // this CTA's (or pair's) place in the tile walk
    const uint32_t nunits = PAIR ? (gridDim.x >> 1) : gridDim.x;
    constexpr int TILE_M = PAIR ? 2 * BM : BM;
    const int64_t tiles_m = (p.M + TILE_M - 1) / TILE_M;
    const int64_t tiles_n = (p.N + BN - 1) / BN;
    const int64_t ntiles = tiles_m * tiles_n;
    const int groups = p.k_iters / 3;                    // slabs per tile: 3 horizontal taps x channel slices
    BNN_CLK_REC(0);
    const int RB = p.b_resident ? NB : 3 * NB;           // barrier pairs of the weight stages

    if (threadIdx.x == 0) {
        // every barrier pair of a ring must have ONE consuming thread (see RingCursor): the slabs alternate between the two
        // issuing threads, so their ring has 2 NA pairs; streamed weight stages change hands every three (one slab's
        // vertical taps), so that ring has RB = 3 NB pairs (NB is even: a multiple of 6 stages and of the NB slots)
        for (int s = 0; s < 2 * NA; ++s) { mbar_init(smem_u32(&ctl->full[s]), 1); mbar_init(smem_u32(&ctl->empty[s]), 1); }
        for (int s = 0; s < RB; ++s) { mbar_init(smem_u32(&ctl->full_b[s]), 1); mbar_init(smem_u32(&ctl->empty_b[s]), 1); }
        for (int b = 0; b < ACC_BUFS; ++b) {
            mbar_init(smem_u32(&ctl->acc_full[b]), N_ISSUE);                          // one commit from each issuing thread
            mbar_init(smem_u32(&ctl->acc_empty[b]), (PAIR ? 2 : 1) * EPI_WARPS);      // the leader's barrier counts both CTAs' warps
        }
        ctl->failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        if (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (PAIR) cluster_sync_all();                        // both CTAs' barriers exist before anyone signals them
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = ctl->tmem_base;

    {   // zero accumulators (every MMA accumulates, see tmem_zero32); unit block scales for the 4-bit instruction (see k_umma_i8)
        if (warp >= 2 && warp < 6) {
            tmem_zero_all(tmem_base, warp, ACC_BUFS * BN);
            if (F4) {
                const uint32_t v = 0x7f7f7f7fu;
                asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1};"
                             ::"r"(tmem_base + SF_COL + ((uint32_t)(32 * (warp & 3)) << 16)), "r"(v) : "memory");
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        if (PAIR) cluster_sync_all();                    // the leader's MMAs write the accumulators and read the scale columns of both CTAs
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    }

    if (warp == 0) {
        // ---------------- TMA producer (in a pair: both CTAs, each its own pixels and its own half of the filters;
        // completion is counted on the leader's "full" barriers, which expect the bytes of both)
        if (lane == 0) {
            bool ok = true;
            const uint32_t tn32 = (uint32_t)tiles_n;
            const uint32_t a_tx = (PAIR ? 2u : 1u) * A_STAGE, b_tx = (PAIR ? 2u : 1u) * B_STAGE;
            auto load_a = [&](uint32_t dst, int c0, int c1, int c2, int c3, uint32_t bar) {
                if (PAIR) tma_load_4d_2sm(dst, &mapA, c0, c1, c2, c3, bar & PEER_MASK);
                else tma_load_4d(dst, &mapA, c0, c1, c2, c3, bar);
            };
            auto load_b = [&](uint32_t dst, int x, int y, uint32_t bar) {
                if (PAIR) tma_load_2d_2sm(dst, &mapB, x, y, bar & PEER_MASK);
                else tma_load_2d(dst, &mapB, x, y, bar);
            };
            const int n_own = (int)(rank * (BN / 2));    // a pair's second CTA keeps the upper half of the tile's filters
            // Resident weights that the preceding kernel did not write are requested before the wait for that kernel.
            bool b_loaded = false;
            if (p.b_resident && p.b_static) {
                const int n0_first = (int)((unit % tn32) * BN) + n_own;
                int kit = 0;
                for (int cc = 0; cc < p.c_chunks; ++cc)
                    for (int dxi = 0; dxi < 3; ++dxi)
                        for (int dyi = 0; dyi < 3; ++dyi, ++kit) {
                            const uint32_t bar = smem_u32(&ctl->full_b[kit]);
                            if (rank == 0) mbar_expect_tx(bar, b_tx);
                            load_b(smem_u32(wts + (size_t)kit * B_STAGE), (3 * dyi + dxi) * p.tap_bytes + cc * KB, n0_first, bar);
                        }
                b_loaded = true;
            }
            bnn_pdl_wait();
            RingCursor ra; ra.start(0, (uint32_t)NA);    // slab ring
            uint32_t sb = 0, bb_i = 0, lapb = 0;         // streamed weights: ring slot, barrier pair, wraps of the barrier ring
            for (uint32_t t = unit; t < (uint32_t)ntiles && ok; t += nunits) {
                const uint32_t tm = t / tn32;
                const int n0 = (int)((t - tm * tn32) * BN) + n_own;
                const int tm128 = PAIR ? 2 * (int)tm + (int)rank : (int)tm;      // this CTA's 128 pixels
                const int tiles_per_img = p.H / p.TH;
                const int b0 = (p.TB > 1) ? tm128 * p.TB : tm128 / tiles_per_img;
                const int y0 = (p.TB > 1) ? 0 : (tm128 % tiles_per_img) * p.TH;
                int kit = 0;
#ifdef BNN_TRACE
                const uint32_t tr_tile = (t - unit) / nunits;
#endif
                for (int cc = 0; cc < p.c_chunks && ok; ++cc) {
                    for (int dxi = 0; dxi < 3 && ok; ++dxi) {
                        if (cc == 0) BNN_TR(0, tr_tile, 2 * dxi);
                        if (ra.reuses((uint32_t)NA) && !mbar_wait(ctl, p.wait_ns, smem_u32(&ctl->empty[ra.prev_bar((uint32_t)NA)]), ra.prev_parity((uint32_t)NA))) { conv_fail<PAIR>(ctl, 21); ok = false; break; }
                        if (cc == 0) BNN_TR(0, tr_tile, 2 * dxi + 1);
                        const uint32_t bar = smem_u32(&ctl->full[ra.b]);
                        if (rank == 0) mbar_expect_tx(bar, a_tx);
                        // dimensions of the map: channel byte, column, image, row
                        load_a(smem_u32(slabs + (size_t)ra.slot((uint32_t)NA) * A_STAGE), cc * KB, dxi - 1, b0, y0 - 1, bar);
                        ra.advance(1, (uint32_t)NA);
                        for (int dyi = 0; dyi < 3; ++dyi, ++kit) {
                            if (p.b_resident) {
                                if (b_loaded) continue;
                                const uint32_t bb = smem_u32(&ctl->full_b[kit]);
                                if (rank == 0) mbar_expect_tx(bb, b_tx);
                                load_b(smem_u32(wts + (size_t)kit * B_STAGE), (3 * dyi + dxi) * p.tap_bytes + cc * KB, n0, bb);
                            } else {
                                if (lapb > 0 || bb_i >= (uint32_t)NB) {      // the stage NB earlier must have been multiplied
                                    const uint32_t pb_i = bb_i >= (uint32_t)NB ? bb_i - (uint32_t)NB : bb_i + (uint32_t)(RB - NB);
                                    const uint32_t pp = (bb_i >= (uint32_t)NB ? lapb : lapb - 1u) & 1u;
                                    if (!mbar_wait(ctl, p.wait_ns, smem_u32(&ctl->empty_b[pb_i]), pp)) { conv_fail<PAIR>(ctl, 22); ok = false; break; }
                                }
                                const uint32_t bb = smem_u32(&ctl->full_b[bb_i]);
                                if (rank == 0) mbar_expect_tx(bb, b_tx);
                                load_b(smem_u32(wts + (size_t)sb * B_STAGE), (3 * dyi + dxi) * p.tap_bytes + cc * KB, n0, bb);
                                if (++sb == (uint32_t)NB) sb = 0;
                                if (++bb_i == (uint32_t)RB) { bb_i = 0; ++lapb; }
                            }
                        }
                    }
                }
                b_loaded = true;
            }
        }
    } else if (warp == 1 || warp == MMA_WARP_B) {
        // ---------------- MMA issuers: two threads (warp 1 and the last warp), alternate SLABS.  What the issuing thread
        // does besides the MMAs themselves -- barrier polls, fences, commits: ~250 clocks per slab -- is not hidden by the
        // tensor pipe's queue, it adds to the pipe's time; with a second thread issuing the next slab's twelve MMAs
        // meanwhile it is.  All products are exact, so the order in which the two streams reach the accumulator does not
        // matter: every MMA accumulates into a buffer that the epilogue left at zero.  In a pair the leader's two threads
        // issue for both tensor cores (M = 256).
        if (lane == 0 && rank == 0) {
            const uint32_t w = (warp == 1) ? 0u : 1u;    // this thread takes the slabs whose running number is w mod 2
            const uint32_t idesc = F4
                ? ((1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | (1u << 23) | ((uint32_t)(TILE_M >> 4) << 24))
                : ((p.idesc & ~(0x1fu << 24)) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24));
            auto mma = [&](uint64_t adesc, uint64_t bdesc, uint32_t tmem_d, uint32_t acc) {
                if (PAIR) { if (F4) umma_mxf4_2sm(tmem_d, adesc, bdesc, idesc, acc, tmem_base + SF_COL); else umma_i8_2sm(tmem_d, adesc, bdesc, idesc, acc); }
                else { if (F4) umma_mxf4(tmem_d, adesc, bdesc, idesc, acc, tmem_base + SF_COL); else umma_i8(tmem_d, adesc, bdesc, idesc, acc); }
            };
            auto commit = [&](uint32_t bar) { if (PAIR) umma_commit_2sm(bar); else umma_commit(bar); };   // in a pair: to both CTAs
            const uint32_t fullA0 = smem_u32(&ctl->full[0]), emptyA0 = smem_u32(&ctl->empty[0]);
            const uint32_t fullB0 = smem_u32(&ctl->full_b[0]), emptyB0 = smem_u32(&ctl->empty_b[0]);
            const uint64_t adesc0 = KB == 64 ? smem_desc_sw64(smem_u32(slabs)) : smem_desc_sw128(smem_u32(slabs));
            const uint64_t bdesc0 = KB == 64 ? smem_desc_sw64(smem_u32(wts)) : smem_desc_sw128(smem_u32(wts));
            const int n_mma = KB >> 5;                   // MMAs (32 bytes of K each) per K step
            const uint32_t a_step = A_STAGE >> 4, b_step = B_STAGE >> 4, dy_step = (uint32_t)p.dy_bytes >> 4;
            uint32_t tc = 0;
            uint32_t j = 0;                              // running number of the tile's first slab (over all tiles of this CTA)
            bool ok = true;
            for (int64_t t = unit; t < ntiles && ok; t += nunits, ++tc, j += (uint32_t)groups) {
                const uint32_t buf = tc & 1;
                const uint32_t tmem_d = tmem_base + buf * BN;
                const bool wait_b = !p.b_resident || tc == 0;
                const uint32_t g_first = (j + w) & 1u;   // first slab of this tile that is this thread's: 0 or 1
                // the accumulator buffer must have been read (and zeroed) by the epilogue of the tile before the last
                if (tc >= ACC_BUFS && !mbar_wait(ctl, p.wait_ns, smem_u32(&ctl->acc_empty[buf]), ((tc / ACC_BUFS) - 1) & 1)) { conv_fail<PAIR>(ctl, 24); ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                BNN_TR(1 + w, tc, 0);
#pragma unroll 1
                for (uint32_t g = g_first; g < (uint32_t)groups && ok; g += 2) {
                    RingCursor ra; ra.start(j + g, (uint32_t)NA);
                    const uint32_t sa = ra.slot((uint32_t)NA);
                    if (!mbar_wait(ctl, p.wait_ns, fullA0 + 8 * ra.b, ra.parity())) { conv_fail<PAIR>(ctl, 26); ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint64_t aslab = adesc0 + (uint64_t)(sa * a_step);
                    const uint32_t kit0 = 3u * g;
                    BNN_TR(1 + w, tc, 1 + g);
#pragma unroll
                    for (uint32_t dyi = 0; dyi < 3; ++dyi) {
                        const uint32_t kit = kit0 + dyi;
                        uint32_t sb = kit, bb_i = kit, pb = 0;       // weight slot, its barrier pair, phase parity
                        if (!p.b_resident) {
                            const uint32_t b_seq = tc * (uint32_t)p.k_iters + kit;
                            sb = b_seq % (uint32_t)NB; bb_i = b_seq % (uint32_t)RB; pb = (b_seq / (uint32_t)RB) & 1u;
                        }
                        if (wait_b) {
                            if (!mbar_wait(ctl, p.wait_ns, fullB0 + 8 * bb_i, pb)) { conv_fail<PAIR>(ctl, 27); ok = false; break; }
                            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        }
                        const uint64_t adesc = aslab + (uint64_t)(dyi * dy_step);
                        const uint64_t bdesc = bdesc0 + (uint64_t)(sb * b_step);
#pragma unroll
                        for (int k = 0; k < BK / 32; ++k) { if (k >= n_mma) break; mma(adesc + 2 * k, bdesc + 2 * k, tmem_d, 1u); }
                        if (!p.b_resident) commit(emptyB0 + 8 * bb_i);
                    }
                    commit(emptyA0 + 8 * ra.b);                 // the slab's three K steps have been issued
                }
                commit(smem_u32(&ctl->acc_full[buf]));          // this thread's share of the tile (also after a failure)
                BNN_TR(1 + w, tc, 11);
            }
        }
    } else if (warp < 2 + EPI_WARPS) {
        // ---------------- epilogue
        bnn_pdl_wait();
        bnn_pdl_launch_next();
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        const int et = threadIdx.x - 64;
        uint32_t tc = 0;
        bool ok = true;
        const uint32_t tn = (uint32_t)tiles_n, nt = (uint32_t)ntiles;
        int64_t n0_prev = -2;                            // filter block whose thresholds the other slot holds
        for (uint32_t t = unit; t < nt; t += nunits, ++tc) {
            const uint32_t buf = tc & 1;
            const uint32_t tm_i = t / tn;
            const int64_t m0 = (int64_t)tm_i * TILE_M + rank * BM, n0 = (int64_t)(t - tm_i * tn) * BN;
            const uint32_t t2 = t + nunits;
            const int64_t n0_next = (t2 < nt) ? (int64_t)(t2 % tn) * BN : -1;
            // the other slot was staged for the tile before this one: with resident weights every tile of a CTA has the same
            // filters, and nothing is fetched or staged after the first two tiles
            epilogue_tile<BN, F4, EPI_WARPS>(ctl, p, tmem_base, buf, tc, m0, n0, n0_next, q, half, lane, et, ok, tc == 0, (tc / ACC_BUFS) & 1, buf ^ 1u,
                                             n0_next == n0_prev);
            n0_prev = n0;
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) { if (PAIR) mbar_arrive_cta0(smem_u32(&ctl->acc_empty[buf])); else mbar_arrive(smem_u32(&ctl->acc_empty[buf])); }
            if (et == 0) BNN_TR(3, tc, 6);
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    BNN_CLK_REC(1);
    if (PAIR) cluster_sync_all();                        // nobody leaves while the partner may still signal its barriers
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}
