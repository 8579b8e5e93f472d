// Decode path for 3 .. 16 tokens on tcgen05/TMEM, scale-MMA form of W^ = L[Q] (.) (BA) with
// 128-column k-steps:
//
//     S      = B_tile (128 x r) * A[:, k-step] (r x 128)        (Eq. 3; bf16 operands, fp32 in TMEM)
//     W^     = L[Q] (.) S                                         (fp16, register -> TMEM)
//     y_tile += W^ (128 x 128) * x[:, k-step]^T (128 x 16)        (fp16 operands, fp32 in TMEM)
//
// It is the memory-bound sibling of the scale-MMA kernel for large token counts: same arithmetic,
// but a k-step of 128 columns (half the barrier traffic per weight element), two main-MMA issuers
// that take k-steps alternately into accumulators of their own, converter warps for the activation
// tile, and a thread-block cluster that splits a tile's k-range and adds the partial sums in the
// leader's shared memory in rank order (deterministic, no atomics).
//
// Warp roles (27 warps):
//   0..15  two worker groups of eight warps take k-steps alternately: a warp owns 32 rows and one
//          64-column half; a thread reads its 64 columns of S from TMEM (as fp16 pairs), looks its code
//          pairs up in a lane-private fp16x2 level table, multiplies and stores W^ straight into TMEM
//          as the A operand.  Group 0 also runs the epilogue.
//   16..19 converters: the activation tile x[16 tokens x 128 columns] arrives as bf16 and is turned
//          into fp16 in place.
//   20,21  main-MMA issuers, one per k-step parity.
//   22,23  scale-MMA issuers, one per k-step parity (= per S buffer).
//   24     TMA producer of the packed code tiles; it also initialises the barriers and starts the
//          weight stream before the rest of the CTA has finished its set-up.
//   25     TMA producer of the B tile (once) and of the factor tiles A[:, k-step].
//   26     TMA producer of the activation tiles.
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

constexpr int kWorkWarps = 16;
constexpr int kGroupWarps = 8;
constexpr int kConvWarp0 = kWorkWarps;                 // 16..19
constexpr int kConvWarps = 4;
constexpr int kIssuerWarp0 = kConvWarp0 + kConvWarps;  // 20, 21
constexpr int kScaleWarp0 = kIssuerWarp0 + 2;          // 22, 23
constexpr int kTmaQWarp = kScaleWarp0 + 2;             // 24
constexpr int kTmaAWarp = kTmaQWarp + 1;               // 25
constexpr int kTmaXWarp = kTmaAWarp + 1;               // 26
constexpr int kWarps = kTmaXWarp + 1;                  // 27
constexpr int kThreads = kWarps * 32;                  // 864
constexpr int kRows = 128;                             // W^ rows per CTA = UMMA M
constexpr int kStep = 128;                             // in-feature columns per k-step
constexpr int kTok = 16;                               // token tile = UMMA N of the main MMA
constexpr int kClusterMax = 8;
constexpr uint32_t kTmemCols = 512;
// TMEM columns: two accumulators (16 each, 32 apart) | S ring (2 x 128 fp32) | W ring (3 x 64)
constexpr uint32_t kSCol = 64;
constexpr int SD = 2;
constexpr uint32_t kWCol = kSCol + SD * kStep;         // 320
constexpr int WS = 3;                                  // W ring = activation ring depth
// A barrier is waited on by parity alone, so whoever waits for its phase n must know that phase n - 1
// has completed: true for a warp that waits for every phase of the barrier, and for a group (or an
// issuer) that owns it.  Worker groups and main issuers take the k-steps alternately, and the W ring
// has an odd depth, so a barrier per W slot would change hands every time round.  The barriers of
// that ring which an alternating role waits on are therefore indexed by the k-step modulo WB, a
// multiple of two: each of them has one owner.
constexpr int WB = 2 * WS;
constexpr int kXAtom = kTok * 128;                     // 16 tokens x 64 columns, 2 bytes each
constexpr int kXStage = 2 * kXAtom;
constexpr int kBTileBytes = kRows * 128;               // B[128 x 64 ranks] bf16

// BITS: code width.  RP: padded rank the factor-tile slots are sized for (32 or 64).
template <int BITS, int RP> struct XCfg {
    static constexpr int QROW = kStep * BITS / 8;              // packed bytes per row per k-step (64 / 48)
    static constexpr int QSTAGE = kRows * QROW;
    static constexpr int SQ = BITS == 4 ? 4 : 6;               // code-tile ring depth (even: one group per barrier)
    static constexpr int AATOM = RP * 128;                     // RP ranks x 64 columns bf16
    // factor-tile ring depth (even: each of its barriers belongs to one scale issuer).  The 4-bit layout keeps
    // this ring below the 64 KB boundary of its level table, where 64 ranks leave room for two stages.
    static constexpr int SA = (BITS == 4 && RP == 64) ? 2 : 4;
    static constexpr int ASTAGE = 2 * AATOM;
    static constexpr int LUT_ENTRIES = BITS == 4 ? 256 : BITS == 3 ? 64 : 16;   // one entry per code pair
    // 32 lane-private copies of every entry (word = lane).  4-bit: entries 256 bytes apart, table on
    // a 64 KB boundary, lookup address by one byte permute; 3- and 2-bit: entries 128 bytes apart,
    // offsets OR-ed into the table-size-aligned base.
    static constexpr int LUT_STRIDE = BITS == 4 ? 256 : 128;
    static constexpr int LUT_BYTES = LUT_ENTRIES * LUT_STRIDE;
    static constexpr int RED_BYTES = kClusterMax * kTok * kRows * 4;   // the cluster's partials, [rank][token][row]
    static constexpr int BAR_BYTES = 512;
    static constexpr int LOW_BYTES = WS * kXStage + kBTileBytes + SA * ASTAGE + BAR_BYTES;   // before the 4-bit table
    static constexpr int SMEM = BITS == 4 ? 232448
                                          : LUT_BYTES /*alignment slack*/ + LUT_BYTES + SQ * QSTAGE + RED_BYTES + LOW_BYTES + 1024;
    static_assert(BITS != 4 || LOW_BYTES + 2048 <= 65536, "4-bit layout: lower part");
    static_assert(BITS != 4 || SQ * QSTAGE + RED_BYTES <= 232448 - 131072, "4-bit layout: upper part");
    static_assert(SMEM <= 232448, "shared memory");
    // barriers
    static constexpr int kBarQFull = 0;                    // SQ: 1 arrival + TMA bytes
    static constexpr int kBarQEmpty = kBarQFull + SQ;      // SQ: the warps of one worker group
    static constexpr int kBarAFull = kBarQEmpty + SQ;      // SA: 1 arrival + TMA bytes
    static constexpr int kBarADone = kBarAFull + SA;       // SA: scale MMA done (commit): frees the factor tile
    static constexpr int kBarXFull = kBarADone + SA;       // WS: 1 arrival + TMA bytes
    static constexpr int kBarXReady = kBarXFull + WS;      // WB: the converter warps
    static constexpr int kBarSFull = kBarXReady + WB;      // SD: scale MMA done (commit)
    static constexpr int kBarSEmpty = kBarSFull + SD;      // SD: the warps of one worker group have read S
    static constexpr int kBarReady = kBarSEmpty + SD;      // WB: the warps of one worker group have written W^
    static constexpr int kBarMmaDone = kBarReady + WB;     // WB: main MMAs of the k-step done (commit): frees W slot and x tile
    static constexpr int kBarAccFull = kBarMmaDone + WB;   // 2: one per main issuer
    static constexpr int kBarReduce = kBarAccFull + 2;     // 1: counts the bytes of the cluster's partial sums
    static constexpr int kBarBFull = kBarReduce + 1;       // 1: 1 arrival + TMA bytes of the B tile
    static constexpr int kBarCount = kBarBFull + 1;
    static_assert(8 * kBarCount + 8 <= BAR_BYTES, "barrier area");
    static_assert(SQ % 2 == 0 && SD % 2 == 0, "one worker group per barrier of these rings");
};

struct alignas(64) Dec16Params {
    CUtensorMap tm_q;     // u8 [m][n*bits/8], box {QROW, 128}
    CUtensorMap tm_a;     // bf16 [r][n], box {64, r_pad}, 128-byte swizzle
    CUtensorMap tm_x;     // bf16 [M][n], box {64, 16}, 128-byte swizzle (rows past M read as zero)
    CUtensorMap tm_b;     // bf16 [m][r], box {64, 128}, 128-byte swizzle (ranks past r read as zero); used if r % 8 == 0
    const uint16_t *B;    // bf16 [m][r]
    float levels[16];
    int M, m, n, r, r_pad;
    int ksteps;           // k-steps per tile
    void *y;
    int y_f32;
    int *status;
    // block-scale instantiation (Eq. 2, the comparator): one scale per row and block of `blk` columns
    const uint16_t *scales;   // bf16 [m][nblk]
    int blk, nblk;
};

// 64 columns of one row: code pairs -> level pairs, times the matching pairs of S (sp, in and out).
// 4-bit rows are 64 bytes and arrive 64-byte-swizzled (16-byte chunk c of row i sits at chunk
// c ^ ((i >> 1) & 3)); 3-bit rows are 48 bytes, pair P at bit 6P of the row's bit stream.
template <int BITS>
__device__ __forceinline__ void dequant_half_row(uint32_t qrow, int row, int ch, uint32_t lut_lane, uint32_t (&sp)[32])
{
    if constexpr (BITS == 4) {
        const uint32_t sw = (uint32_t)((row >> 1) & 3);
        const uint4 c0 = lds_v4(qrow + (((2 * ch) ^ sw) << 4)), c1 = lds_v4(qrow + (((2 * ch + 1) ^ sw) << 4));
        const uint32_t w[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
#pragma unroll
        for (int wi = 0; wi < 8; ++wi)
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const uint32_t lv = lds_u32(__byte_perm(w[wi], lut_lane, 0x7604u | (uint32_t)(b << 4)));
                const __half2 wv = __hmul2(*reinterpret_cast<const __half2 *>(&lv), *reinterpret_cast<const __half2 *>(&sp[wi * 4 + b]));
                sp[wi * 4 + b] = *reinterpret_cast<const uint32_t *>(&wv);
            }
    } else if constexpr (BITS == 2) {
        // 32-byte rows: half ch is the 16 bytes at 16 ch, pair P at bit 4P of them
        const uint4 c0 = lds_v4(qrow + 16 * ch);
        const uint32_t w[4] = {c0.x, c0.y, c0.z, c0.w};
#pragma unroll
        for (int pp = 0; pp < 32; ++pp) {
            const int off = 4 * (pp & 7);
            const uint32_t sh = off >= 7 ? (w[pp >> 3] >> (off - 7)) : (w[pp >> 3] << (7 - off));
            const uint32_t lv = lds_u32((sh & 0x780u) | lut_lane);
            const __half2 wv = __hmul2(*reinterpret_cast<const __half2 *>(&lv), *reinterpret_cast<const __half2 *>(&sp[pp]));
            sp[pp] = *reinterpret_cast<const uint32_t *>(&wv);
        }
    } else {
        // half ch = pairs 32 ch .. 32 ch + 31 = bits 192 ch .. of the 384-bit row = words 6 ch .. 6 ch + 5
        const uint32_t base = qrow + 24 * ch;
        const uint32_t w[6] = {lds_u32(base), lds_u32(base + 4), lds_u32(base + 8), lds_u32(base + 12), lds_u32(base + 16), lds_u32(base + 20)};
#pragma unroll
        for (int pp = 0; pp < 32; ++pp) {
            const int bit = 6 * pp, wi = bit >> 5, off = bit & 31;
            uint32_t sh;
            if (off > 26) sh = __funnelshift_r(w[wi], w[wi + 1 < 6 ? wi + 1 : 5], off - 7);
            else sh = off >= 7 ? (w[wi] >> (off - 7)) : (w[wi] << (7 - off));
            const uint32_t lv = lds_u32((sh & 0x1F80u) | lut_lane);
            const __half2 wv = __hmul2(*reinterpret_cast<const __half2 *>(&lv), *reinterpret_cast<const __half2 *>(&sp[pp]));
            sp[pp] = *reinterpret_cast<const uint32_t *>(&wv);
        }
    }
}

// BLOCK: the scale of an element is its row's block scale (Eq. 2: S = s (x) 1) instead of (BA)_ij: no
// scale MMA, no factor tiles; a worker thread's 64 columns lie in one block (blk is a multiple of 64),
// so its S values are one number read from global memory.  Everything else is the same kernel.
template <int BITS, int RP, bool BLOCK>
__global__ void __launch_bounds__(kThreads, 1) lords_decode16_kernel(const __grid_constant__ Dec16Params p)
{
    using C = XCfg<BITS, RP>;
    constexpr int SQ = C::SQ;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t lut = (raw + C::LUT_BYTES - 1) & ~(uint32_t)(C::LUT_BYTES - 1);   // table-size aligned
    // x0: activation ring; b_tile: B[128 x 64 ranks]; a0: factor ring; q0: code ring;
    // red0: [kClusterMax][16 tokens][128 rows] floats (the leader's copy is used)
    uint32_t x0, b_tile, a0, bars, q0, red0;
    bool fits = true;
    if constexpr (BITS == 4) {
        x0 = (raw + 1023u) & ~1023u;
        b_tile = x0 + WS * kXStage;
        a0 = b_tile + kBTileBytes;
        bars = a0 + C::SA * C::ASTAGE;
        q0 = lut + C::LUT_BYTES;
        red0 = q0 + SQ * C::QSTAGE;
        fits = bars + C::BAR_BYTES <= lut && red0 + C::RED_BYTES <= raw + (uint32_t)C::SMEM;
    } else {
        q0 = lut + C::LUT_BYTES;
        red0 = q0 + SQ * C::QSTAGE;
        x0 = (red0 + C::RED_BYTES + 1023u) & ~1023u;
        b_tile = x0 + WS * kXStage;
        a0 = b_tile + kBTileBytes;
        bars = a0 + C::SA * C::ASTAGE;
        fits = bars + C::BAR_BYTES <= raw + (uint32_t)C::SMEM;
    }
    const uint32_t bar_q_full = bars + 8 * C::kBarQFull, bar_q_empty = bars + 8 * C::kBarQEmpty;
    const uint32_t bar_a_full = bars + 8 * C::kBarAFull, bar_a_done = bars + 8 * C::kBarADone;
    const uint32_t bar_x_full = bars + 8 * C::kBarXFull, bar_x_ready = bars + 8 * C::kBarXReady;
    const uint32_t bar_s_full = bars + 8 * C::kBarSFull, bar_s_empty = bars + 8 * C::kBarSEmpty;
    const uint32_t bar_ready = bars + 8 * C::kBarReady, bar_mma_done = bars + 8 * C::kBarMmaDone;
    const uint32_t bar_acc_full = bars + 8 * C::kBarAccFull, bar_reduce = bars + 8 * C::kBarReduce;
    const uint32_t bar_b_full = bars + 8 * C::kBarBFull;
    const bool b_by_tma = !BLOCK && (p.r & 7) == 0;      // rows of B are 16-byte multiples: the tile comes by TMA
    const uint32_t tmem_slot = bars + 8 * C::kBarCount;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // The cluster shares one tile of 128 rows; rank r takes the r-th slice of its k-steps.
    const int csize = (int)cluster_nctarank(), rank = (int)cluster_ctarank();
    const int tile = (int)blockIdx.x / csize;
    const int row0 = tile * kRows;
    const int ks_a = rank * p.ksteps / csize;          // rank < 8 and ksteps < 2^24: no overflow
    const int ks_b = (rank + 1) * p.ksteps / csize;
    const int total = ks_b - ks_a;

    bool failed = false;
    bool cluster_waited = false;      // this thread has taken the second half of the set-up cluster barrier
    if (!fits) {
        // the shared-memory window does not hold the layout (cannot happen with the window the host
        // asks for; checked because every address below depends on it)
        if (tid == 0) atomicExch(p.status, LORDS_ERR_CUDA);
        return;
    }

    if (warp == kTmaQWarp) {
        // ------------------------------------------------------------------ code tiles (HBM stream)
        // This warp initialises every barrier, releases the rest of the CTA and starts the stream of
        // code tiles at once: the packed codes are weights, nothing in this launch or an earlier one
        // produces them.
        for (int b = lane; b < C::kBarCount; b += 32) {
            uint32_t count = 1;
            if (b >= C::kBarQEmpty && b < C::kBarAFull) count = kGroupWarps;
            else if (b >= C::kBarXReady && b < C::kBarSFull) count = kConvWarps;
            else if (b >= C::kBarSEmpty && b < C::kBarMmaDone) count = kGroupWarps;   // s_empty and ready
            mbar_init(bars + 8 * b, count);
        }
        fence_mbar_init();
        __syncwarp();
        // the leader's reduce barrier counts the bytes of the cluster's partial sums (its one
        // arrival is this one); the stores may come before or after, the phase ends when both are in
        if (rank == 0 && lane == 0 && csize > 1) mbar_expect_tx(bar_reduce, (uint32_t)(csize * kTok * kRows * 4));
        asm volatile("bar.arrive 1, %0;" ::"n"(kThreads) : "memory");   // barriers exist; does not wait for the others
        // split-phase cluster barrier: arrive now (the fence above has published this CTA's barriers
        // cluster-wide, so a relaxed arrival is enough); the wait is in the epilogue
        asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
        if (lane == 0) {
            tma_prefetch_desc(&p.tm_q);
            for (int it = 0; it < total; ++it) {
                const int sq = it % SQ;
                if (it >= SQ) {
                    // a stage is freed by work that stands behind the dependency point: pass it first, so that
                    // the bounded wait does not run while the previous launch (however long) still works
                    if (it == SQ) griddep_wait();
                    if (!mbar_wait(bar_q_empty + 8 * sq, (uint32_t)((it / SQ - 1) & 1))) { failed = true; break; }
                }
                const uint32_t bar = bar_q_full + 8 * sq;
                mbar_expect_tx(bar, (uint32_t)C::QSTAGE);
                tma_load_2d(q0 + sq * C::QSTAGE, &p.tm_q, (ks_a + it) * C::QROW, row0, bar);
            }
        }
    } else {
        if (warp == kIssuerWarp0) {
            tmem_alloc(tmem_slot, kTmemCols);
            tmem_relinquish();
        } else if (warp == kTmaAWarp) {
            if (lane == 0) {
                tma_prefetch_desc(&p.tm_a);
                if (b_by_tma) tma_prefetch_desc(&p.tm_b);
            }
        } else if (warp == kTmaXWarp) {
            if (lane == 0) tma_prefetch_desc(&p.tm_x);
        } else if (warp < kWorkWarps) {
            // level-pair table: entry e = (L[lo code], L[hi code]) as fp16x2; lane's copy of entry e sits
            // at e * LUT_STRIDE + 4 * lane (bank = lane, so the lookups of a warp never conflict)
#pragma unroll
            for (int i = 0; i < C::LUT_ENTRIES / kWorkWarps; ++i) {
                const int entry = warp + kWorkWarps * i;
                const int lo = entry & ((1 << BITS) - 1);
                const int hi = entry >> BITS;
                const __half2 v = __floats2half2_rn(p.levels[lo], p.levels[hi]);
                sts_u32(lut + (uint32_t)(entry * C::LUT_STRIDE + 4 * lane), *reinterpret_cast<const uint32_t *>(&v));
            }
            // B tile: 128 rows x 64 ranks (zero padded) bf16, K-major, 128-byte swizzle: by TMA (below)
            // or, when a row of B is not a multiple of 16 bytes, element by element here
            if (!BLOCK && !b_by_tma && tid < 256) {
                const int rr = tid >> 1, half = tid & 1;
                const int i = row0 + rr;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int chunk = half * 4 + c;
                    uint32_t w4[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int k = chunk * 8 + e * 2;
                        const uint32_t lo = (i < p.m && k < p.r) ? p.B[(size_t)i * p.r + k] : 0u;
                        const uint32_t hi = (i < p.m && k + 1 < p.r) ? p.B[(size_t)i * p.r + k + 1] : 0u;
                        w4[e] = lo | (hi << 16);
                    }
                    sts_v4(b_tile + (rr >> 3) * 1024 + (rr & 7) * 128 + ((chunk ^ (rr & 7)) * 16),
                           make_uint4(w4[0], w4[1], w4[2], w4[3]));
                }
            }
            fence_proxy_async_smem();
        }
        tc_fence_before_sync();
        asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");   // tables, TMEM address and barriers are in place
        tc_fence_after_sync();
        asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");   // see above
    }
    // let a dependent launch (the next layer) begin its own weight prefetch as SMs become free
    griddep_launch_dependents();
    // Everything except the stream of packed codes waits here for the previous launch to finish: a CTA
    // that starts early sets up, prefetches its codes and then stands still, so that every bounded
    // wait below begins behind the dependency point.
    if (warp != kTmaQWarp) griddep_wait();

    if (warp == kTmaQWarp) {
        // all done above
    } else if (warp == kTmaAWarp) {
        // ------------------------------------------------------------------ factor tiles A[:, k-step] (weights)
        if (!BLOCK && lane == 0) {
            if (b_by_tma) {
                mbar_expect_tx(bar_b_full, (uint32_t)kBTileBytes);
                tma_load_2d(b_tile, &p.tm_b, 0, row0, bar_b_full);
            }
            const uint32_t tx = (uint32_t)(2 * p.r_pad * 128);
            for (int it = 0; it < total; ++it) {
                const int sa = it % C::SA;
                if (it >= C::SA && !mbar_wait(bar_a_done + 8 * sa, (uint32_t)((it / C::SA - 1) & 1))) { failed = true; break; }
                const uint32_t bar = bar_a_full + 8 * sa;
                mbar_expect_tx(bar, tx);
#pragma unroll
                for (int at = 0; at < 2; ++at)
                    tma_load_2d(a0 + sa * C::ASTAGE + at * C::AATOM, &p.tm_a, (ks_a + it) * kStep + at * 64, 0, bar);
            }
        }
    } else if (warp == kTmaXWarp) {
        // ------------------------------------------------------------------ activation tiles x[:, k-step]
        if (lane == 0) {
            // x may be the previous launch's output.  (This warp has already waited above with the
            // others; the wait is repeated where the dependency is.)
            griddep_wait();
            for (int it = 0; it < total; ++it) {
                const int sx = it % WS;
                if (it >= WS && !mbar_wait(bar_mma_done + 8 * ((it - WS) % WB), (uint32_t)(((it - WS) / WB) & 1))) { failed = true; break; }
                const uint32_t bar = bar_x_full + 8 * sx;
                mbar_expect_tx(bar, (uint32_t)kXStage);
#pragma unroll
                for (int at = 0; at < 2; ++at)
                    tma_load_2d(x0 + sx * kXStage + at * kXAtom, &p.tm_x, (ks_a + it) * kStep + at * 64, 0, bar);
            }
        }
    } else if (warp >= kScaleWarp0) {
        // ------------------------------------------------------------------ scale-MMA issuers
        // Issuer j takes the k-steps of parity j, i.e. S buffer j.  S of k-step `it` goes into its
        // buffer as soon as the factor tile has landed and the workers have read the buffer's previous content.  One MMA of N = 128 per 16 ranks: its B
        // operand (MN-major) spans the two 64-column atoms of the factor tile, one atom size apart.
        uint32_t tmem_base;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
        constexpr uint32_t idesc_s = umma_idesc_f16(1, 0, 1, kRows, kStep);   // bf16, B operand MN-major, N = 128
        const uint32_t desc_hi = (uint32_t)(umma_desc_sw128(0, 1024, 16) >> 32);
        const uint32_t b_lo = (uint32_t)umma_desc_sw128(0, 1024, 16) | ((b_tile & 0x3FFFFu) >> 4);
        const uint32_t a_lo0 = (uint32_t)umma_desc_sw128(0, 1024, (uint32_t)C::AATOM) | ((a0 & 0x3FFFFu) >> 4);
        const int rsteps = p.r_pad / 16;
        const int sj = warp - kScaleWarp0;
        static_assert(SD == 2 && C::SA % 2 == 0, "one scale issuer per S buffer; each factor-ring barrier belongs to one of them");
        if (b_by_tma && sj < total && !mbar_wait(bar_b_full, 0)) failed = true;
        for (int it = sj; !BLOCK && it < total && !failed; it += 2) {
            const int sa = it % C::SA, sd = it % SD;
            if (!mbar_wait(bar_a_full + 8 * sa, (uint32_t)((it / C::SA) & 1))) { failed = true; break; }
            if (it >= SD && !mbar_wait(bar_s_empty + 8 * sd, (uint32_t)((it / SD - 1) & 1))) { failed = true; break; }
            tc_fence_after_sync();
            if (lane == 0) {
                const uint32_t a_lo = a_lo0 + (uint32_t)(sa * (C::ASTAGE >> 4));
                for (int k = 0; k < rsteps; ++k)
                    umma_f16_ss(tmem_base + kSCol + (uint32_t)(sd * kStep), umma_desc_pack(b_lo + k * 2, desc_hi),
                                umma_desc_pack(a_lo + k * 128, desc_hi), idesc_s, k > 0);
                umma_commit(bar_s_full + 8 * sd);
                umma_commit(bar_a_done + 8 * sa);
            }
            __syncwarp();
        }
    } else if (warp >= kIssuerWarp0) {
        // ------------------------------------------------------------------ main-MMA issuers
        // Issuer j takes the k-steps of parity j into an accumulator of its own (the epilogue adds
        // the two), which doubles the rate at which MMAs leave the CTA.
        const int j = warp - kIssuerWarp0;
        uint32_t tmem_base;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
        constexpr uint32_t idesc_m = umma_idesc_f16(0, 0, 0, kRows, kTok);   // fp16, K-major
        const uint32_t desc_hi = (uint32_t)(umma_desc_sw128(0, 1024, 16) >> 32);
        const uint32_t x_lo0 = (uint32_t)umma_desc_sw128(0, 1024, 16) | ((x0 & 0x3FFFFu) >> 4);
        const uint32_t acc = tmem_base + (uint32_t)(j * 32);
        for (int it = j; it < total; it += 2) {
            const int ws = it % WS;
            if (!mbar_wait(bar_x_ready + 8 * (it % WB), (uint32_t)((it / WB) & 1)) ||
                !mbar_wait(bar_ready + 8 * (it % WB), (uint32_t)((it / WB) & 1))) { failed = true; break; }
            tc_fence_after_sync();
            if (lane == 0) {
                const uint32_t wslot = tmem_base + kWCol + (uint32_t)(ws * 64);
                const uint32_t x_lo = x_lo0 + (uint32_t)(ws * (kXStage >> 4));
#pragma unroll
                for (int k = 0; k < kStep / 16; ++k)
                    umma_f16_ts(acc, wslot + k * 8, umma_desc_pack(x_lo + (k >> 2) * (kXAtom >> 4) + (k & 3) * 2, desc_hi),
                                idesc_m, (it == j && k == 0) ? 0u : 1u);
                umma_commit(bar_mma_done + 8 * (it % WB));
                if (it + 2 >= total) umma_commit(bar_acc_full + 8 * j);
            }
            __syncwarp();
        }
    } else if (warp >= kConvWarp0) {
        // ------------------------------------------------------------------ converters
        // The activation tile (16 tokens x 128 columns bf16, 256 chunks of 16 bytes) becomes fp16 in
        // place: element-wise, so the swizzled position of a chunk does not matter.
        const int ct = (warp - kConvWarp0) * 32 + lane;
        for (int it = 0; it < total; ++it) {
            const int sx = it % WS;
            if (!__all_sync(0xffffffffu, mbar_wait(bar_x_full + 8 * sx, (uint32_t)((it / WS) & 1)))) { failed = true; break; }
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const uint32_t addr = x0 + sx * kXStage + (uint32_t)((c * 128 + ct) * 16);
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
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_x_ready + 8 * (it % WB));
        }
    } else {
        // ------------------------------------------------------------------ worker warps
        // warp wg of a group: lane quadrant q (32 rows), column half ch of the k-step
        const int g = warp / kGroupWarps, wg = warp % kGroupWarps, q = warp & 3, ch = wg >> 2;
        const int row = q * 32 + lane;
        uint32_t tmem_base;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t lut_lane = lut + 4u * (uint32_t)lane;

        for (int it = g; it < total; it += 2) {
            const int sq = it % SQ, sd = it % SD, ws = it % WS;
            // this thread's 64 columns of S, as 32 fp16 pairs
            uint32_t sp[32];
            if constexpr (BLOCK) {
                const int i = row0 + row, blkidx = ((ks_a + it) * kStep + ch * 64) / p.blk;
                const float sc = (i < p.m && blkidx < p.nblk) ? __uint_as_float((uint32_t)p.scales[(size_t)i * p.nblk + blkidx] << 16) : 0.0f;
                const __half2 s2 = __floats2half2_rn(sc, sc);
#pragma unroll
                for (int pp = 0; pp < 32; ++pp) sp[pp] = *reinterpret_cast<const uint32_t *>(&s2);
            } else {
            if (!__all_sync(0xffffffffu, mbar_wait(bar_s_full + 8 * sd, (uint32_t)((it / SD) & 1)))) { failed = true; break; }
            tc_fence_after_sync();
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                uint32_t s[32];
                tmem_ld_32x32(lane_addr + kSCol + (uint32_t)(sd * kStep + ch * 64 + hf * 32), s);
                tmem_wait_ld();
#pragma unroll
                for (int pp = 0; pp < 16; ++pp) {
                    const __half2 sv = __floats2half2_rn(__uint_as_float(s[2 * pp]), __uint_as_float(s[2 * pp + 1]));
                    sp[hf * 16 + pp] = *reinterpret_cast<const uint32_t *>(&sv);
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_s_empty + 8 * sd);      // S is in registers: the buffer may be refilled
            }
            if (!__all_sync(0xffffffffu, mbar_wait(bar_q_full + 8 * sq, (uint32_t)((it / SQ) & 1)))) { failed = true; break; }
            dequant_half_row<BITS>(q0 + sq * C::QSTAGE + row * C::QROW, row, ch, lut_lane, sp);
            // the W slot is free once the MMAs of step it - WS have completed
            if (it >= WS && !__all_sync(0xffffffffu, mbar_wait(bar_mma_done + 8 * ((it - WS) % WB), (uint32_t)(((it - WS) / WB) & 1)))) { failed = true; break; }
            tc_fence_after_sync();
            tmem_st_32x32(lane_addr + kWCol + (uint32_t)(ws * 64 + ch * 32), sp);
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bar_ready + 8 * (it % WB));
                mbar_arrive(bar_q_empty + 8 * sq);
            }
        }

        // Epilogue (group 0, column half 0: one thread per row): the two accumulators -> this CTA's
        // partial y, parked in the cluster leader's shared memory; the leader adds in rank order.
        if (g == 0 && ch == 0 && !failed) {
            const int i = row0 + row;
            // second half of the split-phase cluster barrier, behind the wait for the last MMAs
            if (csize > 1) {
                asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
                cluster_waited = true;
            }
            float yt[kTok];
#pragma unroll
            for (int t = 0; t < kTok; ++t) yt[t] = 0.0f;
            bool ok = true;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                if (ok && j < total) {       // issuer j had a k-step
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_acc_full + 8 * j, 0));
                    tc_fence_after_sync();
                    if (ok) {
                        uint32_t v[16];
                        tmem_ld_32x16(lane_addr + (uint32_t)(j * 32), v);
                        tmem_wait_ld();
#pragma unroll
                        for (int t = 0; t < kTok; ++t) yt[t] += __uint_as_float(v[t]);
                    }
                }
            }
            if (!ok) {
                failed = true;
#pragma unroll
                for (int t = 0; t < kTok; ++t) yt[t] = 0.0f;
            }
            if (csize == 1) {
                if (ok && i < p.m)
#pragma unroll
                    for (int t = 0; t < kTok; ++t)
                        if (t < p.M) store_out(p.y, p.y_f32, (size_t)t * p.m + i, yt[t]);
            } else {
                // a CTA that gave up still sends its bytes (zeros), so the leader never waits in vain
                const uint32_t leader_bar = map_to_rank(bar_reduce, 0);
#pragma unroll
                for (int t = 0; t < kTok; ++t)
                    st_async_cluster_f32(map_to_rank(red0 + (uint32_t)(((rank * kTok + t) * kRows + row) * 4), 0), yt[t], leader_bar);
                if (rank == 0) {
                    const bool got = __all_sync(0xffffffffu, mbar_wait_cluster(bar_reduce, 0));
                    if (!got) failed = true;
                    else if (i < p.m) {
                        // rank order for every token; the sixteen sums run side by side
                        float a[kTok];
#pragma unroll
                        for (int t = 0; t < kTok; ++t) a[t] = 0.0f;
                        for (int rr = 0; rr < csize; ++rr)
#pragma unroll
                            for (int t = 0; t < kTok; ++t)
                                a[t] += __uint_as_float(lds_u32(red0 + (uint32_t)(((rr * kTok + t) * kRows + row) * 4)));
#pragma unroll
                        for (int t = 0; t < kTok; ++t)
                            if (t < p.M) store_out(p.y, p.y_f32, (size_t)t * p.m + i, a[t]);
                    }
                }
            }
        }
    }

    if (failed) atomicExch(p.status, LORDS_ERR_TIMEOUT);
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kIssuerWarp0) {
        tc_fence_after_sync();
        uint32_t tmem_base;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
        tmem_dealloc(tmem_base, kTmemCols);
    }
    // No CTA of the cluster leaves before the leader has received every partial sum: the asynchronous
    // stores of a CTA must not be in flight when it exits (with programmatic dependent launch a CTA
    // of the next launch can take over the SM at once).
    if (csize > 1) {
        // every arrival is paired with a wait: threads that have not waited on the set-up barrier do so first
        if (!cluster_waited) asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
        asm volatile("barrier.cluster.arrive.relaxed;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
    }
}

// One (code width, rank slot) instantiation: launch attributes, resident clusters per size, launch.
template <int BITS, int RP, bool BLOCK> struct Dec16Variant {
    static int prepare(int dev)
    {
        static bool done[kMaxDevices] = {};
        if (!done[dev]) {
            LORDS_CUDA_TRY(cudaFuncSetAttribute(lords_decode16_kernel<BITS, RP, BLOCK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                XCfg<BITS, RP>::SMEM));
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
        cfg.dynamicSmemBytes = XCfg<BITS, RP>::SMEM;
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
            const cudaError_t e = cudaOccupancyMaxActiveClusters(&n, lords_decode16_kernel<BITS, RP, BLOCK>, &cfg);
            if (e != cudaSuccess) (void)cudaGetLastError();
            cache[dev][cs] = (e == cudaSuccess && n >= 1) ? n : -1;
        }
        return cache[dev][cs] > 0 ? cache[dev][cs] : 0;
    }
};

template <int BITS, int RP, bool BLOCK = false> int launch_variant(Dec16Params &k, const Problem &p, const State &st, cudaStream_t stream)
{
    using V = Dec16Variant<BITS, RP, BLOCK>;
    using C = XCfg<BITS, RP>;
    const int dev = device_slot(st), forced_cs = st.forced_splitk;
    int rc = V::prepare(dev);
    if (rc != LORDS_OK) return rc;
    const int tiles = (p.m + kRows - 1) / kRows;
    if (tiles > 65535) return LORDS_ERR_UNSUPPORTED;
    // cluster size: the largest split of the k-range that still lets every cluster be resident at once
    int cs = 1;
    const int lim = kClusterMax < k.ksteps ? kClusterMax : k.ksteps;
    if (forced_cs > 0) {
        cs = forced_cs < lim ? forced_cs : lim;
        while (cs > 1 && V::max_clusters(dev, cs) == 0) --cs;
    } else {
        for (int c = lim; c > 1; --c)
            if (V::max_clusters(dev, c) >= tiles) { cs = c; break; }
    }
    const uint64_t row_bytes = (uint64_t)p.n * BITS / 8;
    if (!make_map_2d(&k.tm_q, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, p.q, row_bytes, (uint64_t)p.m, (uint32_t)C::QROW, (uint32_t)kRows,
                     BITS == 4 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE) ||
        (!BLOCK && !make_map_2d(&k.tm_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p.A, (uint64_t)p.n, (uint64_t)p.r, 64, (uint32_t)k.r_pad,
                                CU_TENSOR_MAP_SWIZZLE_128B)) ||
        !make_map_2d(&k.tm_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p.x, (uint64_t)p.n, (uint64_t)p.M, 64, (uint32_t)kTok,
                     CU_TENSOR_MAP_SWIZZLE_128B))
        return LORDS_ERR_CUDA;
    if (BLOCK) {
        k.tm_a = k.tm_x;      // not used
        k.tm_b = k.tm_x;
    } else if ((p.r & 7) == 0) {
        if (!make_map_2d(&k.tm_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p.B, (uint64_t)p.r, (uint64_t)p.m, 64, (uint32_t)kRows,
                         CU_TENSOR_MAP_SWIZZLE_128B))
            return LORDS_ERR_CUDA;
    } else {
        k.tm_b = k.tm_a;      // not used: the kernel builds the B tile element by element
    }
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    V::fill(cfg, attr, cs, tiles, stream);
    LORDS_CUDA_TRY(cudaLaunchKernelEx(&cfg, lords_decode16_kernel<BITS, RP, BLOCK>, k));
    return LORDS_OK;
}

}  // namespace

// Rules of this path: M <= 16 (with automatic dispatch one or two tokens go to the
// reassociated decode kernel first, and come here when that one declines the rank); r <= 64, which is what the shared-memory layout holds;
// n a multiple of 64 (2- and 4-bit) or 128 (3-bit), which makes every TMA row pitch a multiple of 16 bytes.
// Anything else: LORDS_ERR_UNSUPPORTED.
int launch_decode16(const Problem &p, State &st, cudaStream_t stream)
{
    if (p.bits < 2 || p.bits > 4) return LORDS_ERR_UNSUPPORTED;
    if (p.M > kTok) return LORDS_ERR_UNSUPPORTED;
    if (p.r > 64) return LORDS_ERR_UNSUPPORTED;
    if (p.n % (p.bits == 3 ? 128 : 64) != 0) return LORDS_ERR_UNSUPPORTED;

    Dec16Params k;
    k.B = p.B;
    for (int c = 0; c < 16; ++c) k.levels[c] = p.levels[c];
    k.M = p.M; k.m = p.m; k.n = p.n; k.r = p.r;
    k.r_pad = (p.r + 15) / 16 * 16;
    k.ksteps = (p.n + kStep - 1) / kStep;
    k.y = p.y; k.y_f32 = p.y_f32;
    k.status = st.status_word;
    k.scales = nullptr; k.blk = 0; k.nblk = 0;
    int rc;
    if (p.bits == 4) rc = k.r_pad <= 32 ? launch_variant<4, 32>(k, p, st, stream) : launch_variant<4, 64>(k, p, st, stream);
    else if (p.bits == 3) rc = k.r_pad <= 32 ? launch_variant<3, 32>(k, p, st, stream) : launch_variant<3, 64>(k, p, st, stream);
    else rc = k.r_pad <= 32 ? launch_variant<2, 32>(k, p, st, stream) : launch_variant<2, 64>(k, p, st, stream);
    if (rc != LORDS_OK) return rc;
    st.last_launches = 1;
    st.last_path = "decode16";
    return LORDS_OK;
}

// Block-scale comparator (Eq. 2): y = x (L[Q] (.) (s (x) 1))^T with one bf16 scale per row and block of `blk`
// columns.  Rules: M <= 16; blk a multiple of 64; n a multiple of 64 (2- and 4-bit) or 128 (3-bit).
int launch_blockscale16(const Problem &p, const uint16_t *scales, int blk, State &st, cudaStream_t stream)
{
    if (p.bits < 2 || p.bits > 4) return LORDS_ERR_UNSUPPORTED;
    if (p.M > kTok || blk < 64 || blk % 64 != 0) return LORDS_ERR_UNSUPPORTED;
    if (p.n % (p.bits == 3 ? 128 : 64) != 0) return LORDS_ERR_UNSUPPORTED;
    Dec16Params k;
    k.B = nullptr;
    for (int c = 0; c < 16; ++c) k.levels[c] = p.levels[c];
    k.M = p.M; k.m = p.m; k.n = p.n; k.r = 16;
    k.r_pad = 16;
    k.ksteps = (p.n + kStep - 1) / kStep;
    k.y = p.y; k.y_f32 = p.y_f32;
    k.status = st.status_word;
    k.scales = scales; k.blk = blk; k.nblk = (p.n + blk - 1) / blk;
    const int rc = p.bits == 4 ? launch_variant<4, 32, true>(k, p, st, stream)
                 : p.bits == 3 ? launch_variant<3, 32, true>(k, p, st, stream) : launch_variant<2, 32, true>(k, p, st, stream);
    if (rc != LORDS_OK) return rc;
    st.last_launches = 1;
    st.last_path = "blockscale16";
    return LORDS_OK;
}

}  // namespace lords
