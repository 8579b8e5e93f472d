// Scale-MMA path on tcgen05/TMEM for any token count: W^ = L[Q] (.) (BA) is rebuilt tile by tile.
//
// One CTA owns a 128-row tile of W^ (out-features), a tile of BN tokens and a range of 64-column
// k-steps.  Per k-step:
//   1. TMA brings the factor tile A[r x 64] (bf16) and the activation tile x[BN x 64] into two
//      shared-memory rings of their own (the small factor tiles run ahead of the large activation
//      tiles); the packed code tile Q[128 x 128 columns] comes once per two k-steps;
//   2. the scale issuer runs  S = B_tile (128 x r) * A_tile (r x 64)  (Eq. 3; bf16 operands from
//      shared memory, fp32 result in TMEM) as far ahead of the main MMA as the S ring allows;
//   3. two worker groups of eight warps take the k-steps alternately: a thread reads its 32 columns
//      of S from TMEM, looks its code pairs up in a lane-private fp16x2 level table, forms
//      W^ = L[Q] (.) S in fp16 and stores it straight back into TMEM as the A operand;
//   4. the main issuer runs  D[128 x BN] += W^ (TMEM) * x_tile^T (shared memory), fp32 in TMEM.
// The activations enter the MMA as fp16: for BN = 16 the workers convert the bf16 tile in place,
// for larger token tiles a pre-pass converts x once into scratch.
// Epilogue: D -> registers -> y (bf16 round-to-nearest-even, or fp32).  For BN = 16 the k-range of
// a tile is split over a thread-block cluster whose partial sums meet in the leader's shared
// memory (distributed shared memory) and are added in rank order: deterministic, no atomics.
//
// Every wait is bounded; on expiry the role records LORDS_ERR_TIMEOUT and leaves its loop, so the
// kernel always reaches its final barrier and frees its TMEM.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "lords_internal.h"
#include "lords_ptx.cuh"
#include "lords_tc_common.cuh"

namespace lords {

namespace {

using namespace ptx;

constexpr int BM = 128;                        // W^ rows per CTA = UMMA M
constexpr int BK = 64;                         // in-feature columns per k-step
constexpr int kRMaxUmma = 64;                  // largest rank this path takes (one swizzle atom of K)
constexpr int kWorkWarps = 16;                 // two groups of eight
constexpr int kGroupWarps = 8;
constexpr int kIssuerWarp = kWorkWarps;        // 16: main MMAs
constexpr int kScaleWarp = kWorkWarps + 1;     // 17: scale MMAs, as far ahead as the S ring and the tiles allow
constexpr int kTmaWarp = kWorkWarps + 2;       // 18: activation tiles and code stages
constexpr int kTmaAWarp = kWorkWarps + 3;      // 19: factor tiles
constexpr int kThreads = (kWorkWarps + 4) * 32;   // 640
constexpr int SA = 4;                          // factor-tile ring depth
constexpr int DR = 8;                          // "main MMA of k-step done" barriers, indexed by k-step mod DR
constexpr uint32_t kTmemCols = 512;
constexpr int SQ = 4;                          // code-tile ring depth (128 columns per stage)
constexpr int kBTileBytes = BM * 128;
constexpr int kClusterMax = 8;                 // largest k-split (cluster size) of the BN = 16 kernel

// BITS: code width.  BN: token tile.  RP: padded rank the factor-tile slots are sized for (32 or 64).
template <int BITS, int BN, int RP> struct UCfg {
    static constexpr int QROW = 128 * BITS / 8;                  // packed bytes per row per code stage (64 / 48)
    static constexpr int QSTAGE = BM * QROW;
    // activation ring depth: as deep as shared memory allows, the tiles come from L2 with a latency of
    // several k-steps.  The factor tiles have a ring of their own, so that the scale MMA and the
    // workers run ahead of the (much larger) activation tiles.
    static constexpr int ATILE = RP * 128;
    static constexpr int SX = BN >= 256 ? (RP <= 32 ? 4 : 3) : BN >= 128 ? 6 : 8;
    static constexpr int XTILE = BN * 128;
    // TMEM behind the accumulator is one ring of 64-column slots.  A slot first holds S of a k-step
    // (128 x 64 fp32, written by the scale MMA), then -- in the columns whose S values the writing
    // warp itself has taken into registers -- the fp16 operand W^ of the same k-step, and is free
    // again when the main MMAs of that k-step have completed.  One ring instead of an S ring and a W
    // ring lets the scale MMA run as many k-steps ahead as there are slots.
    static constexpr uint32_t SCOL = BN > 128 ? 256 : 128;       // the ring starts behind the accumulator
    static constexpr int SD = (int)(kTmemCols - SCOL) / 64;      // slots (4 / 6)
    static constexpr int LUT_ENTRIES = BITS == 4 ? 256 : BITS == 3 ? 64 : 16;   // one entry per code pair
    static constexpr int LUT_BYTES = LUT_ENTRIES * 128;
    static constexpr int RED_BYTES = BN == 16 ? kClusterMax * 16 * BM * 4 : 0;
    static constexpr int BAR_BYTES = 512;
    static constexpr int SMEM = 1024 + SX * XTILE + SA * ATILE + SQ * QSTAGE + kBTileBytes + LUT_BYTES + RED_BYTES + BAR_BYTES;
    static constexpr bool kConvertInKernel = BN == 16;           // x tile arrives as bf16 and is converted in place
};

struct alignas(64) UmmaParams {
    CUtensorMap tm_x;     // BN == 16: bf16 [M][n]; else fp16 [M][n]; box {64, BN}, 128-byte swizzle
    CUtensorMap tm_a;     // bf16 [r][n], box {64, r_pad}, 128-byte swizzle
    CUtensorMap tm_q;     // u8 [m][n*bits/8], box {QROW, 128}
    const uint16_t *B;    // bf16 [m][r]
    float levels[16];
    int M, m, n, r, r_pad;
    int npairs;           // 128-column pairs of k-steps per tile
    int tok_tiles;
    int whole_pairs;      // pair mode (BN > 16, clusters of 2): clusters below this index run two whole tiles,
                          // the others share one tile, half of its k-range each; -1 = no pair mode
    float *pair_scratch;  // pair mode: [shared tile][BN][128] partial sums of the second half
    void *y;
    int y_f32;
    int *status;
};

// The 32 columns (chunk c of the 128-column code stage) of one row: codes -> level pairs, times the
// matching pairs of S, as 16 fp16x2 words.
template <int BITS>
__device__ __forceinline__ void dequant_chunk(uint32_t qrow, int row, int c, uint32_t lut_lane, const uint32_t (&s)[32],
                                              uint32_t (&out)[16])
{
    uint32_t lv[16];
    if constexpr (BITS == 4) {
        // 64-byte rows, 64-byte swizzle: 16-byte chunk c of row i sits at chunk c ^ ((i >> 1) & 3)
        const uint4 cw = lds_v4(qrow + (((uint32_t)c ^ (uint32_t)((row >> 1) & 3)) << 4));
        const uint32_t w[4] = {cw.x, cw.y, cw.z, cw.w};
#pragma unroll
        for (int wi = 0; wi < 4; ++wi)
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                // byte b of the word is the code pair: one byte permute isolates it, one multiply-add makes
                // the address of its entry (entries are 128 bytes apart)
                const uint32_t pair = __byte_perm(w[wi], 0u, 0x4440u | (uint32_t)b);
                lv[wi * 4 + b] = lds_u32(lut_lane + pair * 128u);
            }
    } else if constexpr (BITS == 2) {
        // 32-byte rows: chunk c is the 64-bit group at byte 8c; pair p sits at bit 4p of it
        const uint32_t w[2] = {lds_u32(qrow + 8 * c), lds_u32(qrow + 8 * c + 4)};
#pragma unroll
        for (int pp = 0; pp < 16; ++pp) {
            const int off = 4 * (pp & 7);
            const uint32_t sh = off >= 7 ? (w[pp >> 3] >> (off - 7)) : (w[pp >> 3] << (7 - off));
            lv[pp] = lds_u32(lut_lane + (sh & 0x780u));
        }
    } else {
        // 48-byte rows: chunk c is the 96-bit group at byte 12c; pair p sits at bit 6p of it
        const uint32_t w[3] = {lds_u32(qrow + 12 * c), lds_u32(qrow + 12 * c + 4), lds_u32(qrow + 12 * c + 8)};
#pragma unroll
        for (int pp = 0; pp < 16; ++pp) {
            const int bit = 6 * pp, wi = bit >> 5, off = bit & 31;
            uint32_t sh;
            if (off > 26) sh = __funnelshift_r(w[wi], w[wi + 1 < 3 ? wi + 1 : 2], off - 7);
            else sh = off >= 7 ? (w[wi] >> (off - 7)) : (w[wi] << (7 - off));
            lv[pp] = lds_u32(lut_lane + (sh & 0x1F80u));
        }
    }
#pragma unroll
    for (int pp = 0; pp < 16; ++pp) {
        const __half2 sv = __floats2half2_rn(__uint_as_float(s[2 * pp]), __uint_as_float(s[2 * pp + 1]));
        const __half2 wv = __hmul2(*reinterpret_cast<const __half2 *>(&lv[pp]), sv);
        out[pp] = *reinterpret_cast<const uint32_t *>(&wv);
    }
}

template <int BITS, int BN, int RP>
__global__ void __launch_bounds__(kThreads, 1) lords_umma_kernel(const __grid_constant__ UmmaParams p)
{
    using C = UCfg<BITS, BN, RP>;
    constexpr int SX = C::SX, SD = C::SD, kATileBytes = C::ATILE;
    static_assert(DR >= SX && DR >= SD && DR % 2 == 0 && SD % 2 == 0, "done-barrier ring; one worker group per slot");
    static_assert(SD >= SA, "the factor-tile lane frees a tile on the slot barrier of the same k-step");
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    // carve-up (tile bases are multiples of 1024 bytes)
    const uint32_t x0 = base;                                   // SX activation tiles
    const uint32_t a0 = x0 + SX * C::XTILE;                     // SA factor tiles
    const uint32_t q0 = a0 + SA * kATileBytes;                  // SQ code stages
    const uint32_t b_tile = q0 + SQ * C::QSTAGE;                // B[128 x 64 ranks] bf16, K-major, swizzled
    const uint32_t lut = b_tile + kBTileBytes;
    const uint32_t red0 = lut + C::LUT_BYTES;
    const uint32_t bars = red0 + C::RED_BYTES;
    constexpr int kBarXFull = 0;                        // SX: TMA bytes of the activation tile
    constexpr int kBarAFull = kBarXFull + SX;           // SA: TMA bytes of the factor tile
    constexpr int kBarDone = kBarAFull + SA;            // DR: main MMA of the k-step done (commit): frees its x tile and its ring slot
    constexpr int kBarQFull = kBarDone + DR;            // SQ
    constexpr int kBarQEmpty = kBarQFull + SQ;          // SQ: all 16 worker warps (two steps)
    constexpr int kBarSFull = kBarQEmpty + SQ;          // SD: scale MMA done (commit): S is in the slot, the factor tile is free
    constexpr int kBarWFull = kBarSFull + SD;           // SD: one group has written W^ (and converted x)
    constexpr int kBarAccFull = kBarWFull + SD;         // 1
    constexpr int kBarReduce = kBarAccFull + 1;         // 1: the epilogue warps of every CTA of the cluster
    constexpr int kBarCount = kBarReduce + 1;
    static_assert(8 * kBarCount + 8 <= C::BAR_BYTES, "barrier area");
    const uint32_t bar_x_full = bars + 8 * kBarXFull, bar_done = bars + 8 * kBarDone;
    const uint32_t bar_a_full = bars + 8 * kBarAFull;
    const uint32_t bar_q_full = bars + 8 * kBarQFull, bar_q_empty = bars + 8 * kBarQEmpty;
    const uint32_t bar_s_full = bars + 8 * kBarSFull;
    const uint32_t bar_w_full = bars + 8 * kBarWFull;
    const uint32_t bar_acc_full = bars + 8 * kBarAccFull, bar_reduce = bars + 8 * kBarReduce;
    const uint32_t tmem_slot = bars + 8 * kBarCount;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // work assignment: cluster = one (row tile, token tile); rank = slice of its k-range
    const int csize = (int)cluster_nctarank(), rank = (int)cluster_ctarank();
    int tile = (int)blockIdx.x / csize, ksplit = csize, kslice = rank;
    bool pair_split = false;       // this CTA shares its tile with its cluster partner (pair mode)
    int pair_index = 0;
    if (BN > 16 && p.whole_pairs >= 0) {
        // Pair mode fills the idle slots of the last wave: clusters of two CTAs; the first `whole_pairs`
        // clusters run two whole tiles (one per CTA), the remaining clusters split one tile's k-range.
        const int c = (int)blockIdx.x >> 1;
        if (c < p.whole_pairs) {
            tile = 2 * c + rank; ksplit = 1; kslice = 0;
        } else {
            pair_index = c - p.whole_pairs;
            tile = 2 * p.whole_pairs + pair_index; ksplit = 2; kslice = rank; pair_split = true;
        }
    }
    const int row_tile = tile / p.tok_tiles, tok_tile = tile - row_tile * p.tok_tiles;
    const int row0 = row_tile * BM, tok0 = tok_tile * BN;
    const int pa = (int)((long long)kslice * p.npairs / ksplit), pb = (int)((long long)(kslice + 1) * p.npairs / ksplit);
    const int pairs = pb - pa;
    const int total = 2 * pairs;          // k-steps of this CTA; global k-step = 2 * pa + it

    bool failed = false;
    bool cluster_waited = false;      // this thread has taken the second half of the set-up cluster barrier

    if (warp == kTmaWarp) {
        // ------------------------------------------------------------------ TMA producer
        // It also initialises the barriers and starts the weight stream before the rest of the CTA
        // has finished its set-up.
        for (int b = lane; b < kBarCount; b += 32) {
            uint32_t count = 1;
            if (b >= kBarQEmpty && b < kBarSFull) count = kWorkWarps;
            else if (b >= kBarWFull && b < kBarAccFull) count = kGroupWarps;
            else if (b == kBarReduce) count = BN == 16 ? 1u : (uint32_t)(4 * (BN / (BN >= 64 ? BN / 4 : 16)));
            mbar_init(bars + 8 * b, count);
        }
        fence_mbar_init();
        __syncwarp();
        // BN == 16: the leader's reduce barrier counts the bytes of the cluster's partial sums (its one
        // arrival is this one); the stores may come before or after, the phase ends when both are in
        if (BN == 16 && rank == 0 && lane == 0 && csize > 1) mbar_expect_tx(bar_reduce, (uint32_t)(csize * 16 * BM * 4));
        asm volatile("bar.arrive 1, %0;" ::"n"(kThreads) : "memory");   // barriers exist; does not wait for the others
        // split-phase cluster barrier: the fence above has published this CTA's barriers cluster-wide,
        // a relaxed arrival is enough; the wait is in the epilogue before the first remote access
        asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
        if (lane == 0) {
            tma_prefetch_desc(&p.tm_q);
            tma_prefetch_desc(&p.tm_x);
            // Code stages (weights) are issued as early as their ring slot allows: the first SQ at
            // once, later ones whenever a slot is seen free (a non-blocking look), and at the latest --
            // then waiting for the slot -- right before the tiles of the k-steps that need them.
            int next_q = 0;
            auto issue_q = [&](bool blocking) -> bool {
                while (next_q < pairs) {
                    const int sq = next_q % SQ;
                    if (next_q >= SQ) {
                        const uint32_t par = (uint32_t)((next_q / SQ - 1) & 1);
                        if (blocking) {
                            if (!mbar_wait(bar_q_empty + 8 * sq, par)) return false;
                        } else if (!mbar_try_wait(bar_q_empty + 8 * sq, par)) {
                            return true;
                        }
                    }
                    const uint32_t qbar = bar_q_full + 8 * sq;
                    mbar_expect_tx(qbar, (uint32_t)C::QSTAGE);
                    tma_load_2d(q0 + sq * C::QSTAGE, &p.tm_q, (pa + next_q) * C::QROW, row0, qbar);
                    ++next_q;
                    if (blocking) return true;     // one stage was due, no more
                }
                return true;
            };
            issue_q(false);
            // x may be the previous launch's output
            griddep_wait();
            for (int it = 0; it < total; ++it) {
                const int sx = it % SX;
                if (next_q <= (it >> 1) && !issue_q(true)) { failed = true; break; }   // the pair this k-step reads
                if (it >= SX && !mbar_wait(bar_done + 8 * ((it - SX) % DR), (uint32_t)(((it - SX) / DR) & 1))) { failed = true; break; }
                const uint32_t bar = bar_x_full + 8 * sx;
                mbar_expect_tx(bar, (uint32_t)C::XTILE);
                tma_load_2d(x0 + sx * C::XTILE, &p.tm_x, (2 * pa + it) * BK, tok0, bar);
                issue_q(false);
            }
        }
    } else {
        if (warp == kIssuerWarp) {
            tmem_alloc(tmem_slot, kTmemCols);
            tmem_relinquish();
        } else if (warp < kWorkWarps) {
            // level-pair table: entry e = (L[lo code], L[hi code]) as fp16x2; word e*32 + lane is lane's
            // copy (bank = lane, so the lookups of a warp never conflict)
#pragma unroll
            for (int i = 0; i < C::LUT_ENTRIES / kWorkWarps; ++i) {
                const int entry = warp + kWorkWarps * i;
                const int lo = entry & ((1 << BITS) - 1);
                const int hi = entry >> BITS;
                const __half2 v = __floats2half2_rn(p.levels[lo], p.levels[hi]);
                sts_u32(lut + 4u * (uint32_t)(entry * 32 + lane), *reinterpret_cast<const uint32_t *>(&v));
            }
            // B tile: 128 rows x 64 ranks (zero padded) bf16, K-major, 128-byte swizzle
            if (tid < 256) {
                const int rr = tid >> 1, half = tid & 1;
                const int i = row0 + rr;
#pragma unroll
                const bool vec = (p.r & 7) == 0;     // rows of B are 16-byte multiples (B itself is 16-byte aligned)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int chunk = half * 4 + c;
                    uint4 w = make_uint4(0u, 0u, 0u, 0u);
                    if (vec) {
                        if (i < p.m && chunk * 8 < p.r) w = __ldg(reinterpret_cast<const uint4 *>(p.B + (size_t)i * p.r + chunk * 8));
                    } else {
                        uint32_t w4[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int k = chunk * 8 + e * 2;
                            const uint32_t lo = (i < p.m && k < p.r) ? p.B[(size_t)i * p.r + k] : 0u;
                            const uint32_t hi = (i < p.m && k + 1 < p.r) ? p.B[(size_t)i * p.r + k + 1] : 0u;
                            w4[e] = lo | (hi << 16);
                        }
                        w = make_uint4(w4[0], w4[1], w4[2], w4[3]);
                    }
                    sts_v4(b_tile + (rr >> 3) * 1024 + (rr & 7) * 128 + ((chunk ^ (rr & 7)) * 16), w);
                }
            }
            fence_proxy_async_smem();
        }
        tc_fence_before_sync();
        asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");   // tables, TMEM address and barriers are in place
        tc_fence_after_sync();
        asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
    }
    // let a dependent launch begin its own weight prefetch as SMs become free
    griddep_launch_dependents();

    if (warp == kTmaWarp) {
        // all done above
    } else if (warp == kTmaAWarp) {
        // ------------------------------------------------------------------ factor tiles (weights)
        if (lane == 0) {
            tma_prefetch_desc(&p.tm_a);
            const uint32_t tx = (uint32_t)(p.r_pad * 128);
            for (int j = 0; j < total; ++j) {
                const int sa = j % SA;
                // the tile's slot is free once the scale MMA of k-step j - SA has completed: that is the
                // commit the workers wait for as well (this lane looks at every phase of those barriers
                // in turn, and no slot barrier can run a phase ahead of it: the scale MMA of k-step
                // j - SA + SD needs a factor tile that this lane has not loaded yet)
                if (j >= SA && !mbar_wait(bar_s_full + 8 * ((j - SA) % SD), (uint32_t)(((j - SA) / SD) & 1))) { failed = true; break; }
                const uint32_t bar = bar_a_full + 8 * sa;
                mbar_expect_tx(bar, tx);
                tma_load_2d(a0 + sa * kATileBytes, &p.tm_a, (2 * pa + j) * BK, 0, bar);
            }
        }
    } else if (warp == kScaleWarp) {
        // ------------------------------------------------------------------ scale-MMA issuer
        // S of k-step j goes into ring slot j % SD as soon as the factor tile has landed and the main MMAs
        // of k-step j - SD are done with the slot: it runs SD k-steps ahead of the main MMAs by itself.
        uint32_t tmem_base;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
        constexpr uint32_t idesc_s = umma_idesc_f16(1, 0, 1, BM, 64);     // bf16, B operand MN-major, N = 64
        const uint32_t desc_hi = (uint32_t)(umma_desc_sw128(0, 1024, 16) >> 32);
        const uint32_t lbo_lo = (uint32_t)umma_desc_sw128(0, 1024, 16);
        const uint32_t b_lo = lbo_lo | ((b_tile & 0x3FFFFu) >> 4);
        const uint32_t a_lo0 = lbo_lo | ((a0 & 0x3FFFFu) >> 4);
        const int ksteps = p.r_pad / 16;
        for (int j = 0; j < total; ++j) {
            const int sa = j % SA, sd = j % SD;
            if (!mbar_wait(bar_a_full + 8 * sa, (uint32_t)((j / SA) & 1))) { failed = true; break; }
            // the slot is free once the main MMAs of k-step j - SD have read their operand out of it
            if (j >= SD && !mbar_wait(bar_done + 8 * ((j - SD) % DR), (uint32_t)(((j - SD) / DR) & 1))) { failed = true; break; }
            tc_fence_after_sync();
            if (lane == 0) {
                const uint32_t a_lo = a_lo0 + (uint32_t)(sa * (kATileBytes >> 4));
                for (int k = 0; k < ksteps; ++k)
                    umma_f16_ss(tmem_base + C::SCOL + sd * 64, umma_desc_pack(b_lo + k * 2, desc_hi),
                                umma_desc_pack(a_lo + k * 128, desc_hi), idesc_s, k > 0);
                umma_commit(bar_s_full + 8 * sd);
            }
            __syncwarp();
        }
    } else if (warp == kIssuerWarp) {
        // ------------------------------------------------------------------ main-MMA issuer
        uint32_t tmem_base;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
        constexpr uint32_t idesc_m = umma_idesc_f16(0, 0, 0, BM, BN);     // fp16, K-major
        const uint32_t desc_hi = (uint32_t)(umma_desc_sw128(0, 1024, 16) >> 32);
        const uint32_t x_lo0 = (uint32_t)umma_desc_sw128(0, 1024, 16) | ((x0 & 0x3FFFFu) >> 4);
        for (int it = 0; it < total; ++it) {
            const int sx = it % SX, ws = it % SD;
            // W^ of the k-step is in TMEM and its activation tile has landed
            if (!mbar_wait(bar_w_full + 8 * ws, (uint32_t)((it / SD) & 1))) { failed = true; break; }
            if (!mbar_wait(bar_x_full + 8 * sx, (uint32_t)((it / SX) & 1))) { failed = true; break; }
            tc_fence_after_sync();
            if (lane == 0) {
                const uint32_t wslot = tmem_base + C::SCOL + (uint32_t)(ws * 64);
                const uint32_t x_lo = x_lo0 + (uint32_t)((sx * C::XTILE) >> 4);
#pragma unroll
                for (int k = 0; k < BK / 16; ++k)
                    // columns 0-31 of the k-step sit in slot columns 0-15, columns 32-63 in 32-47
                    umma_f16_ts(tmem_base, wslot + (k >> 1) * 32 + (k & 1) * 8, umma_desc_pack(x_lo + k * 2, desc_hi), idesc_m,
                                (it > 0 || k > 0) ? 1u : 0u);
                umma_commit(bar_done + 8 * (it % DR));
                if (it == total - 1) umma_commit(bar_acc_full);
            }
            __syncwarp();
        }
    } else {
        // ------------------------------------------------------------------ worker warps
        const int g = warp / kGroupWarps, wg = warp % kGroupWarps, q = warp & 3, ch = wg >> 2;
        const int row = q * 32 + lane;
        uint32_t tmem_base;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t lut_lane = lut + 4u * (uint32_t)lane;

        for (int it = g; it < total; it += 2) {
            const int sx = it % SX, sd = it % SD, pr = it >> 1, sq = pr % SQ;
            if (!__all_sync(0xffffffffu, mbar_wait(bar_s_full + 8 * sd, (uint32_t)((it / SD) & 1)))) { failed = true; break; }
            tc_fence_after_sync();
            uint32_t s[32];
            tmem_ld_32x32(lane_addr + C::SCOL + (uint32_t)(sd * 64 + ch * 32), s);
            bool ok = mbar_wait(bar_q_full + 8 * sq, (uint32_t)((pr / SQ) & 1));
            tmem_wait_ld();
            if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
            uint32_t out[16];
            dequant_chunk<BITS>(q0 + sq * C::QSTAGE + row * C::QROW, row, (it & 1) * 2 + ch, lut_lane, s, out);
            if constexpr (C::kConvertInKernel) {
                // The activation tile arrived as bf16 (16 tokens x 64 columns): convert it in place, one 16-byte chunk per
                // thread of the first four warps of the group (element-wise, so the swizzled position
                // of the chunk does not matter).
                if (!__all_sync(0xffffffffu, mbar_wait(bar_x_full + 8 * sx, (uint32_t)((it / SX) & 1)))) { failed = true; break; }
                if (wg < 4) {
                    const uint32_t addr = x0 + sx * C::XTILE + (uint32_t)((wg * 32 + lane) * 16);
                    const uint4 v = lds_v4(addr);
                    const uint32_t in[4] = {v.x, v.y, v.z, v.w};
                    uint32_t o[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const __half2 hv = __floats2half2_rn(__uint_as_float(in[e] << 16), __uint_as_float(in[e] & 0xFFFF0000u));
                        o[e] = *reinterpret_cast<const uint32_t *>(&hv);
                    }
                    sts_v4(addr, make_uint4(o[0], o[1], o[2], o[3]));
                }
                fence_proxy_async_smem();
            }
            // W^ goes where this warp's own S values were: nobody else reads those columns of these lanes
            tmem_st_32x16(lane_addr + C::SCOL + (uint32_t)(sd * 64 + ch * 32), out);
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bar_w_full + 8 * sd);
                mbar_arrive(bar_q_empty + 8 * sq);
            }
        }

        // ------------------------------------------------------------------ epilogue
        constexpr int CPG = BN >= 64 ? BN / 4 : 16;      // accumulator columns per warp column group
        const int cg = warp >> 2;
        if (cg * CPG < BN && !failed) {
            bool ok = true;
            // BN == 16, k-range split over the cluster: the second half of the split-phase cluster barrier
            // (every CTA has initialised its barriers) is taken here, behind the wait for the last MMAs
            if (BN == 16 && csize > 1) {
                asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
                cluster_waited = true;
            }
            if (total > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar_acc_full, 0));
            tc_fence_after_sync();
            const int i = row0 + row;
            if (!ok) failed = true;
            if (BN > 16 || csize == 1) {
                float *const part = p.pair_scratch + (size_t)pair_index * BN * BM;
                if (pair_split && rank == 0) {
                    // the partner's half of the k-range comes through global scratch; its arrival on
                    // this CTA's barrier (release / acquire at cluster scope) orders the data
                    if (!__all_sync(0xffffffffu, mbar_wait_cluster(bar_reduce, 0))) { ok = false; failed = true; }
                }
                if (ok && total > 0) {
#pragma unroll 1
                    for (int c0 = cg * CPG; c0 < (cg + 1) * CPG; c0 += 16) {
                        uint32_t v[16];
                        tmem_ld_32x16(lane_addr + (uint32_t)c0, v);
                        tmem_wait_ld();
                        if (pair_split && rank == 1) {
#pragma unroll
                            for (int c = 0; c < 16; ++c) part[(size_t)(c0 + c) * BM + row] = __uint_as_float(v[c]);
                        } else if (i < p.m) {
                            // the partner's sums of the chunk are all requested before the first store to y (which
                            // the compiler must assume may alias them: load and store by turns would pay the way to
                            // L2 sixteen times)
                            float pv[16];
#pragma unroll
                            for (int c = 0; c < 16; ++c) pv[c] = pair_split ? __ldcg(part + (size_t)(c0 + c) * BM + row) : 0.0f;
#pragma unroll
                            for (int c = 0; c < 16; ++c) {
                                const int t = tok0 + c0 + c;
                                if (t < p.M) store_out(p.y, p.y_f32, (size_t)t * p.m + i, __uint_as_float(v[c]) + pv[c]);   // fixed order: first half + second half
                            }
                        }
                    }
                }
                if (pair_split && rank == 1) {
                    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");   // the partner's barrier exists
                    cluster_waited = true;
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(map_to_rank(bar_reduce, 0));
                }
            } else {
                // BN == 16 with the k-range split over the cluster: park the partials in the leader's
                // shared memory; a CTA that gave up still arrives (with zeros)
                uint32_t v[16];
#pragma unroll
                for (int c = 0; c < 16; ++c) v[c] = 0u;
                if (ok && total > 0) {
                    tmem_ld_32x16(lane_addr, v);
                    tmem_wait_ld();
                }
                const uint32_t leader_bar = map_to_rank(bar_reduce, 0);
#pragma unroll
                for (int c = 0; c < 16; ++c)
                    st_async_cluster_f32(map_to_rank(red0 + (uint32_t)(((rank * 16 + c) * BM + row) * 4), 0), __uint_as_float(v[c]), leader_bar);
                if (rank == 0) {
                    if (!__all_sync(0xffffffffu, mbar_wait_cluster(bar_reduce, 0))) failed = true;
                    else if (i < p.m) {
#pragma unroll 1
                        for (int c = 0; c < 16; ++c) {
                            const int t = tok0 + c;
                            if (t >= p.M) break;
                            float a = 0.0f;
                            for (int rr = 0; rr < csize; ++rr)
                                a += __uint_as_float(lds_u32(red0 + (uint32_t)(((rr * 16 + c) * BM + row) * 4)));
                            store_out(p.y, p.y_f32, (size_t)t * p.m + i, a);
                        }
                    }
                }
            }
        }
    }

    if (failed) atomicExch(p.status, LORDS_ERR_TIMEOUT);
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kIssuerWarp) {
        tc_fence_after_sync();
        uint32_t tmem_base;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
        tmem_dealloc(tmem_base, kTmemCols);
    }
    // Clusters (split k-range of the 16-token tile, or a pair): no CTA leaves before its partner has
    // received what it sent (asynchronous stores and remote arrivals of a CTA must not be in flight
    // when it exits)
    if (csize > 1) {
        // every arrival is paired with a wait: threads that have not waited on the set-up barrier do so first
        if (!cluster_waited) asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
        asm volatile("barrier.cluster.arrive.relaxed;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
    }
}

// x bf16 -> fp16 (exact for every bf16 value inside fp16's normal range), 8 elements per thread.
__global__ void lords_x_to_f16_kernel(const uint4 *__restrict__ x, uint4 *__restrict__ x16, size_t n_vec, int early)
{
    // Programmatic dependent launch on both sides (early != 0): the kernel that consumes x16 may begin its
    // set-up (weights only) at once; this kernel itself waits for the previous launch, which may still be
    // writing x or reading the scratch that x16 overwrites.  (Without the launch attribute both are no-ops.)
    if (early) griddep_launch_dependents();
    griddep_wait();
    size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n_vec) return;
    const uint4 v = x[e];
    const uint32_t in[4] = {v.x, v.y, v.z, v.w};
    uint32_t out[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float lo = __uint_as_float(in[q] << 16);
        const float hi = __uint_as_float(in[q] & 0xFFFF0000u);
        const __half2 h = __floats2half2_rn(lo, hi);
        out[q] = *reinterpret_cast<const uint32_t *>(&h);
    }
    x16[e] = make_uint4(out[0], out[1], out[2], out[3]);
}

template <int BITS, int BN, int RP> struct UmmaVariant {
    static int prepare(int dev)
    {
        static bool done[kMaxDevices] = {};
        if (!done[dev]) {
            LORDS_CUDA_TRY(cudaFuncSetAttribute(lords_umma_kernel<BITS, BN, RP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                UCfg<BITS, BN, RP>::SMEM));
            done[dev] = true;
        }
        return LORDS_OK;
    }
    static void fill(cudaLaunchConfig_t &cfg, cudaLaunchAttribute *attr, int cs, int clusters, cudaStream_t stream)
    {
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)cs;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        // programmatic dependent launch: the kernel touches only weights until its griddepcontrol.wait
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg = cudaLaunchConfig_t{};
        cfg.gridDim = dim3((unsigned)(clusters * cs));
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = UCfg<BITS, BN, RP>::SMEM;
        cfg.stream = stream;
        cfg.attrs = attr;
        cfg.numAttrs = 2;
    }
    // Clusters of `cs` CTAs that can be resident at the same time (0 if such a cluster cannot run).
    static int max_clusters(int dev, int cs)
    {
        static int cache[kMaxDevices][kClusterMax + 1];   // 0 = not asked yet, -1 = cannot run
        if (cache[dev][cs] == 0) {
            cudaLaunchConfig_t cfg;
            cudaLaunchAttribute attr[2];
            fill(cfg, attr, cs, 1, nullptr);
            int n = 0;
            const cudaError_t e = cudaOccupancyMaxActiveClusters(&n, lords_umma_kernel<BITS, BN, RP>, &cfg);
            if (e != cudaSuccess) (void)cudaGetLastError();
            cache[dev][cs] = (e == cudaSuccess && n >= 1) ? n : -1;
        }
        return cache[dev][cs] > 0 ? cache[dev][cs] : 0;
    }
    static int launch(const UmmaParams &k, int tiles, int cs, cudaStream_t stream)
    {
        cudaLaunchConfig_t cfg;
        cudaLaunchAttribute attr[2];
        fill(cfg, attr, cs, tiles, stream);
        LORDS_CUDA_TRY(cudaLaunchKernelEx(&cfg, lords_umma_kernel<BITS, BN, RP>, k));
        return LORDS_OK;
    }
};

template <int BITS, int BN, int RP> int launch_variant(UmmaParams &k, const Problem &p, State &st, cudaStream_t stream)
{
    using V = UmmaVariant<BITS, BN, RP>;
    const int dev = device_slot(st);
    int rc = V::prepare(dev);
    if (rc != LORDS_OK) return rc;
    k.tok_tiles = (p.M + BN - 1) / BN;
    const int row_tiles = (p.m + BM - 1) / BM;
    const long long tiles = (long long)row_tiles * k.tok_tiles;
    if (tiles > 0x3fffffffLL) return LORDS_ERR_UNSUPPORTED;

    // k-split over a cluster: only the BN = 16 kernel has the shared-memory reduction
    int cs = 1;
    if (BN == 16) {
        const bool forced = st.forced_splitk > 0;
        const long long want = forced ? st.forced_splitk : st.sm_count / tiles;
        int lim = want < kClusterMax ? (int)want : kClusterMax;
        if (lim > k.npairs) lim = k.npairs;
        for (int c = lim; c > 1; --c)
            if (V::max_clusters(dev, c) >= (forced ? 1 : tiles)) { cs = c; break; }
    }

    // Pair mode (BN > 16): when the tiles need more than one wave of CTAs, idle slots of the last wave
    // are filled by splitting that many tiles' k-range over the two CTAs of a cluster; when the tiles
    // fill at most half of the resident CTAs, every tile's k-range is split (a tile is a serial chain
    // of k-steps, so half the range is half the time).
    k.whole_pairs = -1;
    k.pair_scratch = nullptr;
    int clusters = (int)tiles;
    size_t pair_bytes = 0;
    if (BN > 16 && k.npairs >= 2) {
        const long long resident = 2LL * V::max_clusters(dev, 2);
        if (resident > 0 && tiles > resident) {
            const long long waves = (tiles + resident - 1) / resident;
            long long split = waves * resident - tiles;
            if (split > tiles) split = tiles;
            if ((tiles - split) & 1) --split;
            if (split > 0) {
                k.whole_pairs = (int)((tiles - split) / 2);
                clusters = k.whole_pairs + (int)split;
                cs = 2;
                pair_bytes = (size_t)split * BN * BM * sizeof(float);
            }
        } else if (resident > 0 && 2 * tiles <= resident) {
            k.whole_pairs = 0;
            clusters = (int)tiles;
            cs = 2;
            pair_bytes = (size_t)tiles * BN * BM * sizeof(float);
        }
    }

    const void *xsrc = p.x;
    if (!UCfg<BITS, BN, RP>::kConvertInKernel) {
        const size_t x16_bytes = ((size_t)p.M * p.n * 2 + 255) & ~(size_t)255;
        if (x16_bytes + pair_bytes > st.workspace_bytes) return LORDS_ERR_WORKSPACE;
        k.pair_scratch = reinterpret_cast<float *>(st.workspace + x16_bytes);
        const size_t n_vec = (size_t)p.M * p.n / 8;
        // A short pre-pass overlaps the main kernel's set-up (-2 us per call at 512 tokens); next to a long one
        // (2048 tokens x 14336 columns: 18 us at the HBM rate) the early main kernel's CTAs and weight prefetch
        // cost more than the overlap gains (+2 us), so there the main kernel starts when the pre-pass is done.
        const int early = (size_t)p.M * p.n <= ((size_t)8 << 20) ? 1 : 0;
        cudaLaunchAttribute pre_attr[1];
        pre_attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        pre_attr[0].val.programmaticStreamSerializationAllowed = early;
        cudaLaunchConfig_t pre_cfg = cudaLaunchConfig_t{};
        pre_cfg.gridDim = dim3((unsigned)((n_vec + 255) / 256));
        pre_cfg.blockDim = dim3(256);
        pre_cfg.stream = stream;
        pre_cfg.attrs = pre_attr;
        pre_cfg.numAttrs = 1;
        LORDS_CUDA_TRY(cudaLaunchKernelEx(&pre_cfg, lords_x_to_f16_kernel, reinterpret_cast<const uint4 *>(p.x),
                                          reinterpret_cast<uint4 *>(st.workspace), n_vec, early));
        xsrc = st.workspace;
    }
    const uint64_t row_bytes = (uint64_t)p.n * BITS / 8;
    if (!make_map_2d(&k.tm_x, UCfg<BITS, BN, RP>::kConvertInKernel ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16,
                     2, xsrc, (uint64_t)p.n, (uint64_t)p.M, 64, (uint32_t)BN, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_2d(&k.tm_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p.A, (uint64_t)p.n, (uint64_t)p.r, 64, (uint32_t)k.r_pad,
                     CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_2d(&k.tm_q, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, p.q, row_bytes, (uint64_t)p.m, (uint32_t)UCfg<BITS, BN, RP>::QROW, BM,
                     BITS == 4 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE))
        return LORDS_ERR_CUDA;
    rc = V::launch(k, clusters, cs, stream);
    if (rc != LORDS_OK) return rc;
    st.last_launches = UCfg<BITS, BN, RP>::kConvertInKernel ? 1 : 2;
    return LORDS_OK;
}

template <int BITS, int RP> int launch_bits_rank(UmmaParams &k, const Problem &p, State &st, cudaStream_t stream)
{
    if (p.M <= 16) return launch_variant<BITS, 16, RP>(k, p, st, stream);
    // token tile: the largest that still gives CTAs for most of the SMs (tiles that fill at most half of the
    // SMs are split over two CTAs each, see launch_variant)
    const long long row_tiles = (p.m + BM - 1) / BM;
    auto ctas = [&](int b) {
        const long long t = row_tiles * ((p.M + b - 1) / b);
        return (2 * t <= st.sm_count && p.n > 128) ? 2 * t : t;
    };
    int bn = 256;
    while (bn > 32 && (p.M <= bn / 2 || 5 * ctas(bn) < 3 * (long long)st.sm_count)) bn /= 2;
    if (st.forced_bn > 0) bn = st.forced_bn;   // measurement switch
    switch (bn) {
        case 32: return launch_variant<BITS, 32, RP>(k, p, st, stream);
        case 64: return launch_variant<BITS, 64, RP>(k, p, st, stream);
        case 128: return launch_variant<BITS, 128, RP>(k, p, st, stream);
        default: return launch_variant<BITS, 256, RP>(k, p, st, stream);
    }
}

template <int BITS> int launch_bits(UmmaParams &k, const Problem &p, State &st, cudaStream_t stream)
{
    return k.r_pad <= 32 ? launch_bits_rank<BITS, 32>(k, p, st, stream) : launch_bits_rank<BITS, 64>(k, p, st, stream);
}

}  // namespace

// Rules of this path: r <= 64; n a multiple of 64 (2- and 4-bit codes) or 128 (3-bit), which makes
// every TMA row pitch a multiple of 16 bytes.  Anything else: LORDS_ERR_UNSUPPORTED.
int launch_umma(const Problem &p, State &st, cudaStream_t stream)
{
    if (p.bits < 2 || p.bits > 4) return LORDS_ERR_UNSUPPORTED;
    if (p.r > kRMaxUmma || p.n % (p.bits == 3 ? 128 : 64) != 0) return LORDS_ERR_UNSUPPORTED;

    UmmaParams k;
    k.B = p.B;
    for (int c = 0; c < 16; ++c) k.levels[c] = p.levels[c];
    k.M = p.M; k.m = p.m; k.n = p.n; k.r = p.r;
    k.r_pad = (p.r + 15) / 16 * 16;
    k.npairs = (p.n + 127) / 128;
    k.y = p.y; k.y_f32 = p.y_f32;
    k.status = st.status_word;
    const int rc = p.bits == 4 ? launch_bits<4>(k, p, st, stream) : p.bits == 3 ? launch_bits<3>(k, p, st, stream) : launch_bits<2>(k, p, st, stream);
    if (rc != LORDS_OK) return rc;
    st.last_path = "umma";
    return LORDS_OK;
}

}  // namespace lords
