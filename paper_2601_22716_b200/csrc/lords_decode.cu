// Decode path (M <= 2 tokens) on tcgen05/TMEM, reassociated form of W^ = L[Q] (.) (BA):
//
//     z[t][i][k] = sum_j L[Q_ij] * (A_kj * x_tj)          (one GEMM, N = M * r columns)
//     y[t][i]    = sum_k B_ik * z[t][i][k]                 (a row dot product in the epilogue)
//
// which equals y = x (L[Q] (.) (BA))^T with S = BA of Eq. 3 never formed: the scale factors
// ride on the small operand, so the big operand is the bare level table lookup of the codes.
//
// A thread-block cluster owns one tile of 128 * H rows of Q (H = 1 or 2); its CTAs split the tile's
// k-steps (128 in-feature columns each) evenly, and the host picks H and the cluster size so that
// all clusters are resident at once and fill the SMs.  Each CTA sends its partial y into the cluster
// leader's shared memory with asynchronous stores whose bytes the leader's mbarrier counts; the
// leader adds the partials in rank order -- deterministic, no float atomics, no trip through
// global memory.  A cluster barrier at the very end keeps every CTA alive until the leader is done.
//
// Warp roles (28 warps):
//   0..15  two worker groups of eight warps take k-steps alternately and dequantise: a warp owns 32
//          rows (H = 2: all 128 columns of the k-step; H = 1: one 64-column half); a thread reads its
//          row's packed codes from shared memory, looks every code pair up in a lane-private fp16x2
//          level table and stores the levels straight into TMEM as the A operand (tcgen05.st).
//          Group 0 also runs the epilogue.
//   16..23 two converter groups of four warps take k-steps alternately: they turn the factor tile
//          A[:, k-step] (TMA, shared memory) in place into the fp16 B operand A_kj * x_tj.
//   24,25  MMA issuers: D[128 x N] += W[128 x 16] * AX[N x 16]^T with A from TMEM and B from shared
//          memory, eight per k-step; one issuer per 128-row half (H = 2) or per k-step parity (H = 1).
//   26     TMA producer of the packed code tiles (HBM stream, deep ring); it also initialises the
//          barriers and starts the stream before the rest of the CTA has finished its set-up.
//   27     TMA producer of the factor tiles and of the k-step's slice of x (two tensor maps, one barrier).
//
// Every wait is bounded; on expiry the role records LORDS_ERR_TIMEOUT and leaves its loop, so
// the kernel always reaches its final barrier and frees its TMEM.  The waits carry tags for the
// diagnostic record of the first wait that ran out: 1 code stage free, 2 factor stage free, 3 B operand
// written, 4 W slot written, 5 factor tile and x landed, 6 W slot free, 7 code tile landed,
// 8 accumulator complete, 9 partial sums received.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <type_traits>

#include "lords_internal.h"
#include "lords_ptx.cuh"
#include "lords_tc_common.cuh"

namespace lords {

namespace {

using namespace ptx;

constexpr int kWorkWarps = 16;                         // worker warps: two groups of eight
constexpr int kConvWarp0 = kWorkWarps;                 // 16..23: converters of the factor tiles
constexpr int kConvGroupWarps = 4;
constexpr int kConvGroups = 2;
constexpr int kIssuerWarp0 = kConvWarp0 + kConvGroups * kConvGroupWarps;   // 24, 25: one per half (H == 2) or per k-step parity (H == 1)
constexpr int kTmaQWarp = kIssuerWarp0 + 2;            // 26
constexpr int kTmaAWarp = kTmaQWarp + 1;               // 27
constexpr int kWarps = kTmaAWarp + 1;                  // 28
constexpr int kThreads = kWarps * 32;                  // 896
constexpr int kNMax = 64;                              // accumulator columns per half (N = M * r_pad)
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kWCol = 2 * kNMax;                  // W ring starts behind the accumulators
constexpr int kAtomBytes = kNMax * 128;                // one 64-column swizzle atom of the B operand
constexpr int kClusterMax = 16;                        // largest cluster (split of a tile's k-range) this kernel is launched with
constexpr int kStep = 128;                             // in-feature columns per k-step
constexpr int kAtoms = kStep / 64;
constexpr int kWSlotCols = kStep / 2;                  // TMEM columns of one W slot (fp16 pairs)

// BITS: code width.  H: 128-row halves per CTA tile (1 or 2).
template <int BITS, int H> struct DCfg {
    static constexpr int TILE_ROWS = 128 * H;
    static constexpr int GROUP_WARPS = 8;                      // worker warps on one k-step
    static constexpr int GROUPS = kWorkWarps / GROUP_WARPS;    // two groups take k-steps alternately
    static constexpr int COLS = kStep * H / 2;                 // columns of the k-step one thread dequantises (64 / 128)
    static constexpr int QROW = kStep * BITS / 8;              // packed bytes per row per k-step (64 / 48)
    static constexpr int QSTAGE = TILE_ROWS * QROW;
    static constexpr int SQ = (BITS == 4 ? 8 : 12) / H;        // code-tile ring depth: 64 / 72 KB in flight
    static constexpr int S_TMEM = (512 - (int)kWCol) / (H * kWSlotCols);
    static constexpr int S = S_TMEM < 4 ? S_TMEM : 4;          // W / factor ring depth (4 / 3)
    static constexpr int AXSTAGE = kAtoms * kAtomBytes;
    static constexpr int XSTAGE = 2 * kStep * 2;               // the k-step's slice of x, two tokens (bf16)
    static constexpr int LUT_ENTRIES = BITS == 4 ? 256 : BITS == 3 ? 64 : 16;   // one entry per code pair
    // 32 lane-private copies of every entry (word = lane, so the lookups of a warp never conflict).
    // 4-bit: an entry every 256 bytes and the table on a 64 KB boundary, which lets one byte
    // permute build a lookup address: byte 0 = 4 * lane, byte 1 = the code pair's byte, bytes 2..3 =
    // the table's base.  3- and 2-bit: an entry every 128 bytes, offsets OR-ed into the table-size-aligned base.
    static constexpr int LUT_STRIDE = BITS == 4 ? 256 : 128;
    static constexpr int LUT_BYTES = LUT_ENTRIES * LUT_STRIDE;
    static constexpr int RED_BYTES = kClusterMax * 2 * TILE_ROWS * 4;   // the cluster's partials, [rank][token][row]
    static constexpr int BAR_BYTES = 512;
    // 4-bit: the buffers are laid out around the table, some before its 64 KB boundary, the rest
    // behind it, inside the largest shared-memory window a CTA can have; AX_LOW of the factor stages
    // sit in the lower part
    static constexpr int AX_LOW = BITS == 4 ? (H == 1 ? 2 : 1) : S;
    static constexpr int SMEM = BITS == 4 ? 232448
                                          : LUT_BYTES /*alignment slack*/ + LUT_BYTES + SQ * QSTAGE + S * (AXSTAGE + XSTAGE) + RED_BYTES + BAR_BYTES;
    // the code ring's depth is a multiple of the group count, so each of its barriers is used by
    // one group alone, which then sees every phase of it
    static_assert(SQ % GROUPS == 0, "code ring depth must be a multiple of the group count");
};

struct alignas(64) DecodeParams {
    CUtensorMap tm_q;     // u8 [m][n*bits/8], box {QROW, 128 * H}
    CUtensorMap tm_a;     // bf16 [r][n], box {64, r_pad}, 128-byte swizzle
    CUtensorMap tm_x;     // bf16 [M][n], box {128, M}, no swizzle (columns past n read as zero)
    const uint16_t *x;    // bf16 [M][n]
    const uint16_t *B;    // bf16 [m][r]
    float levels[16];
    int M, m, n, r, r_pad;
    int ksteps;           // k-steps per tile
    int tiles;
    void *y;
    int y_f32;
    int *status;
};

// One row of one k-step (128 codes): packed codes (shared memory) -> fp16 level pairs -> 64 TMEM columns.
// 4-bit rows are 64 bytes and arrive 64-byte-swizzled (16-byte chunk c of row i sits at chunk
// c ^ ((i >> 1) & 3)), which spreads the 16-byte reads of eight consecutive rows over all banks;
// 3-bit rows are 48 bytes, a stride that is conflict-free as it is.
template <int BITS, int COLS>
__device__ __forceinline__ void dequant_row_to_tmem(uint32_t qrow, int row, int ch, uint32_t lut_lane, uint32_t taddr)
{
    // COLS == 128: the thread does the whole row (two 64-column halves); COLS == 64: only half `ch`.
    constexpr int kHalves = COLS / 64;
    if constexpr (BITS == 4) {
        const uint32_t sw = (uint32_t)((row >> 1) & 3);
#pragma unroll
        for (int hh = 0; hh < kHalves; ++hh) {
            const int half = kHalves == 2 ? hh : ch;
            const uint4 c0 = lds_v4(qrow + (((2 * half) ^ sw) << 4)), c1 = lds_v4(qrow + (((2 * half + 1) ^ sw) << 4));
            const uint32_t w[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
            uint32_t out[32];
#pragma unroll
            for (int wi = 0; wi < 8; ++wi)
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    // byte b of the word holds two codes, its entry sits at byte * 256: the address is
                    // the table's lane address with that byte as byte 1
                    out[wi * 4 + b] = lds_u32(__byte_perm(w[wi], lut_lane, 0x7604u | (uint32_t)(b << 4)));
                }
            tmem_st_32x32(taddr + half * 32, out);
        }
    } else if constexpr (BITS == 2) {
        // 32-byte rows: half h is the 16 bytes at 16 h, code pair P at bit 4P of them
#pragma unroll
        for (int hh = 0; hh < kHalves; ++hh) {
            const int half = kHalves == 2 ? hh : ch;
            const uint4 c0 = lds_v4(qrow + 16 * half);
            const uint32_t w[4] = {c0.x, c0.y, c0.z, c0.w};
            uint32_t out[32];
#pragma unroll
            for (int pp = 0; pp < 32; ++pp) {
                const int off = 4 * (pp & 7);
                const uint32_t sh = off >= 7 ? (w[pp >> 3] >> (off - 7)) : (w[pp >> 3] << (7 - off));
                out[pp] = lds_u32((sh & 0x780u) | lut_lane);
            }
            tmem_st_32x32(taddr + half * 32, out);
        }
    } else {
        const uint4 c0 = lds_v4(qrow), c1 = lds_v4(qrow + 16), c2 = lds_v4(qrow + 32);
        const uint32_t w[12] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w, c2.x, c2.y, c2.z, c2.w};
        auto half_row = [&](auto half_c) {
            constexpr int half = decltype(half_c)::value;
            uint32_t out[32];
#pragma unroll
            for (int pp = 0; pp < 32; ++pp) {
                // code pair P sits at bit 6P of the row's 384-bit little-endian stream
                const int bit = 6 * (half * 32 + pp), wi = bit >> 5, off = bit & 31;
                uint32_t sh;
                if (off > 26) sh = __funnelshift_r(w[wi], w[wi + 1 < 12 ? wi + 1 : 11], off - 7);
                else sh = off >= 7 ? (w[wi] >> (off - 7)) : (w[wi] << (7 - off));
                out[pp] = lds_u32((sh & 0x1F80u) | lut_lane);
            }
            tmem_st_32x32(taddr + half * 32, out);
        };
        if (kHalves == 2 || ch == 0) half_row(std::integral_constant<int, 0>{});
        if (kHalves == 2 || ch == 1) half_row(std::integral_constant<int, 1>{});
    }
}

template <int BITS, int NTOK, int H>
__global__ void __launch_bounds__(kThreads, 1) lords_decode_kernel(const __grid_constant__ DecodeParams p)
{
    using C = DCfg<BITS, H>;
    constexpr int S = C::S, SQ = C::SQ, kTileRows = C::TILE_ROWS, kGroups = C::GROUPS, kGroupWarps = C::GROUP_WARPS;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t lut = (raw + C::LUT_BYTES - 1) & ~(uint32_t)(C::LUT_BYTES - 1);   // table-size aligned
    // q0: code ring; ax_lo / ax_hi: factor stages 0 .. AX_LOW-1 and AX_LOW .. S-1 (tile bases are
    // multiples of 1024); xs0: x slices of the k-steps in flight, [stage][token][128] bf16;
    // red0: [kClusterMax][NTOK][rows] floats, the cluster's partials (leader's copy is used)
    constexpr int kAxLow = C::AX_LOW;
    uint32_t q0, ax_lo, ax_hi, xs0, red0, bars;
    bool fits = true;
    if constexpr (BITS == 4) {
        ax_lo = (raw + 1023u) & ~1023u;
        xs0 = ax_lo + kAxLow * C::AXSTAGE;
        red0 = xs0 + ((S * C::XSTAGE + 1023) & ~1023);
        bars = red0 + C::RED_BYTES;
        q0 = lut + C::LUT_BYTES;
        ax_hi = q0 + SQ * C::QSTAGE;
        fits = bars + C::BAR_BYTES <= lut && ax_hi + (S - kAxLow) * C::AXSTAGE <= raw + (uint32_t)C::SMEM;
    } else {
        q0 = lut + C::LUT_BYTES;
        ax_lo = q0 + SQ * C::QSTAGE;
        ax_hi = ax_lo;
        xs0 = ax_lo + S * C::AXSTAGE;
        red0 = xs0 + S * C::XSTAGE;
        bars = red0 + C::RED_BYTES;
    }
    auto ax_stage = [&](int s) -> uint32_t {
        return s < kAxLow ? ax_lo + (uint32_t)(s * C::AXSTAGE) : ax_hi + (uint32_t)((s - kAxLow) * C::AXSTAGE);
    };
    // mbarriers, 8 bytes each, in one run so that a warp can initialise them lane-parallel
    constexpr int kBarQFull = 0;                            // SQ, 1 arrival + TMA bytes
    constexpr int kBarQEmpty = kBarQFull + SQ;              // SQ, the warps of one group
    // A barrier is waited on by parity alone, so whoever waits for its phase n must know that phase
    // n - 1 has completed.  A warp that waits for every phase of a barrier knows; so does a group that
    // owns the barrier.  The converter groups take the k-steps alternately: with an odd ring depth a
    // stage would change hands every time round, and a group that polls "stage s, second filling"
    // while the first filling (the other group's) is still in flight would see the phase it waits
    // for as already complete.  The "factor tile landed" barriers are therefore indexed by the k-step
    // modulo a multiple of the group count, which gives every barrier one owner; so are the "MMAs of
    // the k-step done" barriers, which the worker groups wait on alternately.
    constexpr int kAF = S % kConvGroups == 0 ? S : S * kConvGroups;
    constexpr int kBarAFull = kBarQEmpty + SQ;              // kAF, 1 arrival + TMA bytes
    constexpr int kBarAxReady = kBarAFull + kAF;            // S: the warps of one converter group (B operand written)
    constexpr int kBarReady = kBarAxReady + S;              // H * S: the warps of one worker group (W slot written)
    constexpr int kBarMmaDone = kBarReady + H * S;          // kAF, one commit per half
    constexpr int kBarAccFull = kBarMmaDone + kAF;          // 2: one per issuer
    constexpr int kBarReduce = kBarAccFull + 2;             // 1: counts the bytes of the cluster's partial sums (leader's copy is used)
    constexpr int kBarCount = kBarReduce + 1;
    static_assert(8 * kBarCount + 8 <= C::BAR_BYTES, "barrier area");
    static_assert(SQ % kGroups == 0, "one worker group per code-ring barrier");
    const uint32_t bar_q_full = bars + 8 * kBarQFull, bar_q_empty = bars + 8 * kBarQEmpty;
    const uint32_t bar_a_full = bars + 8 * kBarAFull, bar_ax_ready = bars + 8 * kBarAxReady, bar_ready = bars + 8 * kBarReady;
    const uint32_t bar_mma_done = bars + 8 * kBarMmaDone, bar_acc_full = bars + 8 * kBarAccFull;
    const uint32_t bar_reduce = bars + 8 * kBarReduce;
    const uint32_t tmem_slot = bars + 8 * kBarCount;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // The cluster shares one tile of 128 * H rows; rank r takes the r-th slice of its k-steps.
    const int csize = (int)cluster_nctarank(), rank = (int)cluster_ctarank();
    const int tile = (int)blockIdx.x / csize;
    const int ks_a = rank * p.ksteps / csize;          // rank < 16 and ksteps < 2^24: no overflow
    const int ks_b = (rank + 1) * p.ksteps / csize;
    const int total = ks_b - ks_a;
    const int N = NTOK * p.r_pad;
    const int *status = p.status;

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
        for (int b = lane; b < kBarCount; b += 32) {
            uint32_t count = 1;
            if (b >= kBarQEmpty && b < kBarAFull) count = kGroupWarps;
            else if (b >= kBarAxReady && b < kBarReady) count = kConvGroupWarps;
            else if (b >= kBarReady && b < kBarMmaDone) count = kGroupWarps / H;   // the warps that fill this half's W slot
            else if (b >= kBarMmaDone && b < kBarAccFull) count = H;   // H == 1: the step's one issuer
            mbar_init(bars + 8 * b, count);
        }
        fence_mbar_init();
        __syncwarp();
        // the leader's reduce barrier counts the bytes of the cluster's partial sums (its one
        // arrival is this one); the stores may come before or after, the phase ends when both are in
        if (rank == 0 && lane == 0 && csize > 1) mbar_expect_tx(bar_reduce, (uint32_t)(csize * NTOK * kTileRows * 4));
        asm volatile("bar.arrive 1, %0;" ::"n"(kThreads) : "memory");   // barriers exist; does not wait for the others
        // split-phase cluster barrier: arrive now (this CTA's reduce barrier exists and the fence above
        // has published it cluster-wide, so a relaxed arrival is enough); the wait is in the epilogue,
        // right before the first access to the leader's shared memory
        asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
        if (lane == 0) {
            tma_prefetch_desc(&p.tm_q);
            for (int it = 0; it < total; ++it) {
                const int sq = it % SQ;
                if (it >= SQ) {
                    // a stage is freed by work that stands behind the dependency point: pass it first, so that
                    // the bounded wait does not run while the previous launch (however long) still works
                    if (it == SQ) griddep_wait();
                    if (!mbar_wait(bar_q_empty + 8 * sq, (uint32_t)((it / SQ - 1) & 1), status, 1)) { failed = true; break; }
                }
                const uint32_t bar = bar_q_full + 8 * sq;
                mbar_expect_tx(bar, (uint32_t)C::QSTAGE);
                tma_load_2d(q0 + sq * C::QSTAGE, &p.tm_q, (ks_a + it) * C::QROW, tile * kTileRows, bar);
            }
        }
    } else {
        if (warp == kIssuerWarp0) {
            tmem_alloc(tmem_slot, kTmemCols);
            tmem_relinquish();
        } else if (warp == kTmaAWarp) {
            if (lane == 0) {
                tma_prefetch_desc(&p.tm_a);
                tma_prefetch_desc(&p.tm_x);
            }
        } else if (warp < kWorkWarps) {
            // level-pair table: entry e = (L[lo code], L[hi code]) as fp16x2; word e*32 + lane is lane's
            // copy (bank = lane, so the lookups of a warp never conflict)
            // warp w writes entries w, w + 16, ...; the loads of the levels are independent
#pragma unroll
            for (int i = 0; i < C::LUT_ENTRIES / kWorkWarps; ++i) {
                const int entry = warp + kWorkWarps * i;
                const int lo = entry & ((1 << BITS) - 1);
                const int hi = entry >> BITS;
                const __half2 v = __floats2half2_rn(p.levels[lo], p.levels[hi]);
                sts_u32(lut + (uint32_t)(entry * C::LUT_STRIDE + 4 * lane), *reinterpret_cast<const uint32_t *>(&v));
            }
        }
        tc_fence_before_sync();
        asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");   // table, TMEM address and barriers are in place
        tc_fence_after_sync();
        asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");   // see above
    }
    // let a dependent launch (the next layer) begin its own weight prefetch as SMs become free
    griddep_launch_dependents();
    // Everything except the two streams of weights (packed codes, first factor tiles) waits here for
    // the previous launch to finish: a CTA that starts early sets up, prefetches and then stands still,
    // so every bounded wait below begins behind the dependency point.
    if (warp != kTmaQWarp && warp != kTmaAWarp) griddep_wait();

    if (warp == kTmaQWarp) {
        // all done above
    } else if (warp == kTmaAWarp) {
        // ------------------------------------------------------------------ factor tiles A[:, k-step] and x[:, k-step]
        if (lane == 0) {
            const uint32_t tx_a = (uint32_t)(kAtoms * p.r_pad * 128);
            // one barrier per stage counts the bytes of the factor tile and of the x slice
            auto load_a = [&](int it) {
                const int s = it % S, j0 = (ks_a + it) * kStep;
                const uint32_t bar = bar_a_full + 8 * (it % kAF);
                mbar_expect_tx(bar, tx_a + (uint32_t)(NTOK * kStep * 2));
#pragma unroll
                for (int at = 0; at < kAtoms; ++at)
                    tma_load_2d(ax_stage(s) + at * kAtomBytes, &p.tm_a, j0 + at * 64, 0, bar);
            };
            auto load_x = [&](int it) {
                const int s = it % S;
                tma_load_2d(xs0 + s * C::XSTAGE, &p.tm_x, (ks_a + it) * kStep, 0, bar_a_full + 8 * (it % kAF));
            };
            // the factors are weights: the first stages are filled before the dependency point
            const int pre = total < S ? total : S;
            for (int it = 0; it < pre; ++it) load_a(it);
            griddep_wait();   // x may be the previous launch's output
            for (int it = 0; it < pre; ++it) load_x(it);
            for (int it = S; it < total; ++it) {
                if (!mbar_wait(bar_mma_done + 8 * ((it - S) % kAF), (uint32_t)(((it - S) / kAF) & 1), status, 2)) { failed = true; break; }
                load_a(it);
                load_x(it);
            }
        }
    } else if (warp >= kIssuerWarp0) {
        // ------------------------------------------------------------------ MMA issuers
        // H == 2: issuer j owns half j and takes every k-step.  H == 1: the two issuers take the
        // k-steps alternately, each into its own accumulator (the epilogue adds the two), which
        // doubles the rate at which MMAs leave the CTA.
        const int j = warp - kIssuerWarp0;
        const int h = H == 2 ? j : 0;
        constexpr int kStride = H == 2 ? 1 : 2;
        static_assert(H == 2 || S % 2 == 0, "with alternating issuers every ring barrier belongs to one of them");
        uint32_t tmem_base;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
        const uint32_t idesc = (1u << 4) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);  // fp16 x fp16 -> fp32, K-major
        const uint32_t desc_hi = (uint32_t)(umma_desc_sw128(0, 1024, 16) >> 32);
        const uint32_t desc_lo = (uint32_t)umma_desc_sw128(0, 1024, 16);
        const uint32_t acc = tmem_base + (uint32_t)(j * kNMax);
        const int first = H == 2 ? 0 : j;
        for (int it = first; it < total; it += kStride) {
            const int s = it % S;
            if (!mbar_wait(bar_ax_ready + 8 * s, (uint32_t)((it / S) & 1), status, 3) ||
                !mbar_wait(bar_ready + 8 * (h * S + s), (uint32_t)((it / S) & 1), status, 4)) { failed = true; break; }
            tc_fence_after_sync();
            if (lane == 0) {
                const uint32_t wslot = tmem_base + kWCol + (uint32_t)((h * S + s) * kWSlotCols);
                const uint32_t b_lo = desc_lo | ((ax_stage(s) & 0x3FFFFu) >> 4);
#pragma unroll
                for (int k = 0; k < kStep / 16; ++k)
                    umma_f16_ts(acc, wslot + k * 8, umma_desc_pack(b_lo + (k >> 2) * (kAtomBytes >> 4) + (k & 3) * 2, desc_hi),
                                idesc, (it == first && k == 0) ? 0u : 1u);
                umma_commit(bar_mma_done + 8 * (it % kAF));
                if (it + kStride >= total) umma_commit(bar_acc_full + 8 * j);
            }
            __syncwarp();
        }
    } else if (warp >= kConvWarp0) {
        // ------------------------------------------------------------------ converters
        // B operand: A_kj * x_tj as fp16, in place (token 0) and behind it (token 1).  A lane owns the
        // 16-byte chunk c16 (8 columns) of rows rsub + kRowStep * i of both 64-column atoms.
        const int cgp = (warp - kConvWarp0) / kConvGroupWarps, cw = (warp - kConvWarp0) % kConvGroupWarps;
        const int c16 = lane & 7, rsub = cw * 4 + (lane >> 3);
        constexpr int kRowStep = 4 * kConvGroupWarps;          // 16
        constexpr int kRowIters = kNMax / kRowStep;            // 4
        for (int it = cgp; it < total; it += kConvGroups) {
            const int s = it % S;
            if (!__all_sync(0xffffffffu, mbar_wait(bar_a_full + 8 * (it % kAF), (uint32_t)((it / kAF) & 1), status, 5))) { failed = true; break; }
#pragma unroll
            for (int at = 0; at < kAtoms; ++at) {
                const uint32_t atom = ax_stage(s) + at * kAtomBytes;
                uint4 av[kRowIters];
#pragma unroll
                for (int i = 0; i < kRowIters; ++i) {
                    const int k = rsub + kRowStep * i;
                    if (k < p.r_pad) av[i] = lds_v4(atom + k * 128 + ((c16 ^ (k & 7)) << 4));
                }
                float xf[NTOK][8];
#pragma unroll
                for (int t = 0; t < NTOK; ++t) {
                    // columns past n were filled with zeros by the tensor-map copy
                    const uint4 xv = lds_v4(xs0 + s * C::XSTAGE + t * (kStep * 2) + at * 128 + c16 * 16);
                    const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        xf[t][2 * e] = __uint_as_float(xw[e] << 16);
                        xf[t][2 * e + 1] = __uint_as_float(xw[e] & 0xFFFF0000u);
                    }
                }
#pragma unroll
                for (int i = 0; i < kRowIters; ++i) {
                    const int k = rsub + kRowStep * i;
                    if (k < p.r_pad) {
                        const uint32_t addr = atom + k * 128 + ((c16 ^ (k & 7)) << 4);
                        const uint32_t aw4[4] = {av[i].x, av[i].y, av[i].z, av[i].w};
#pragma unroll
                        for (int t = 0; t < NTOK; ++t) {
                            uint32_t o[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const __half2 hv = __floats2half2_rn(__uint_as_float(aw4[e] << 16) * xf[t][2 * e],
                                                                     __uint_as_float(aw4[e] & 0xFFFF0000u) * xf[t][2 * e + 1]);
                                o[e] = *reinterpret_cast<const uint32_t *>(&hv);
                            }
                            sts_v4(addr + t * p.r_pad * 128, make_uint4(o[0], o[1], o[2], o[3]));
                        }
                    }
                }
            }
            // the stores above become visible to the tensor core's (async-proxy) reads
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_ax_ready + 8 * s);
        }
    } else {
        // ------------------------------------------------------------------ worker warps
        // warp wg of a group: lane quadrant q; H == 2: row half h, all 128 columns of the k-step;
        // H == 1: the one row half, column half ch
        const int g = warp / kGroupWarps, wg = warp % kGroupWarps, q = warp & 3;
        const int h = H == 2 ? (wg >> 2) : 0, ch = H == 2 ? 0 : (wg >> 2);
        const int row_in_tile = h * 128 + q * 32 + lane;
        uint32_t tmem_base;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t lut_lane = lut + 4u * (uint32_t)lane;

        for (int it = g; it < total; it += kGroups) {
            const int sq = it % SQ, s = it % S;
            // the W slot is free once the MMAs of step it - S have completed
            if (it >= S && !__all_sync(0xffffffffu, mbar_wait(bar_mma_done + 8 * ((it - S) % kAF), (uint32_t)(((it - S) / kAF) & 1), status, 6))) { failed = true; break; }
            tc_fence_after_sync();

            // codes -> levels -> TMEM
            if (!__all_sync(0xffffffffu, mbar_wait(bar_q_full + 8 * sq, (uint32_t)((it / SQ) & 1), status, 7))) { failed = true; break; }
            dequant_row_to_tmem<BITS, C::COLS>(q0 + sq * C::QSTAGE + row_in_tile * C::QROW, row_in_tile, ch, lut_lane,
                                      lane_addr + kWCol + (uint32_t)((h * S + s) * kWSlotCols));
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bar_ready + 8 * (h * S + s));
                mbar_arrive(bar_q_empty + 8 * sq);
            }
        }

        // Epilogue (group 0): z (TMEM) . B row -> this CTA's partial y, parked in the cluster
        // leader's shared memory; the leader adds the cluster's partials in rank order.
        if (g == 0 && ch == 0) {
            const int i = tile * kTileRows + row_in_tile;
            // B row first, so its latency hides behind the wait for the last MMAs
            uint4 bq[kNMax / 8];
            if ((p.r & 7) == 0) {
#pragma unroll
                for (int c = 0; c < kNMax / 8; ++c)
                    bq[c] = (i < p.m && c * 8 < p.r) ? __ldg(reinterpret_cast<const uint4 *>(p.B + (size_t)i * p.r) + c)
                                                     : make_uint4(0, 0, 0, 0);
            } else {
                // ranks that are not a multiple of 8: the rows of B are not 16-byte aligned
#pragma unroll
                for (int c = 0; c < kNMax / 8; ++c) {
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int k = c * 8 + 2 * e;
                        const uint32_t lo = (i < p.m && k < p.r) ? __ldg(p.B + (size_t)i * p.r + k) : 0u;
                        const uint32_t hi = (i < p.m && k + 1 < p.r) ? __ldg(p.B + (size_t)i * p.r + k + 1) : 0u;
                        w[e] = lo | (hi << 16);
                    }
                    bq[c] = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
            // second half of the split-phase cluster barrier (every CTA of the cluster has initialised
            // its barriers): taken here, where its latency hides behind the wait for the last MMAs
            if (csize > 1) {
                asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
                cluster_waited = true;
            }
            float yt[NTOK];
#pragma unroll
            for (int t = 0; t < NTOK; ++t) yt[t] = 0.0f;
            bool ok = !failed;
            // H == 2: this half's accumulator.  H == 1: the accumulators of both issuers (the second
            // one only if it had a k-step at all).
            constexpr int kAccs = H == 2 ? 1 : 2;
#pragma unroll
            for (int a = 0; a < kAccs; ++a) {
                const int j = H == 2 ? h : a;
                if (ok && j < total + (H == 2 ? 2 : 0)) {
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_acc_full + 8 * j, 0, status, 8));
                    tc_fence_after_sync();
                    if (ok) {
#pragma unroll
                        for (int t = 0; t < NTOK; ++t) {
                            float acc = yt[t];
#pragma unroll
                            for (int c = 0; c < kNMax / 16; ++c) {
                                if (c * 16 < p.r_pad) {   // warp-uniform
                                    uint32_t v[16];
                                    tmem_ld_32x16(lane_addr + (uint32_t)(j * kNMax + t * p.r_pad + c * 16), v);
                                    tmem_wait_ld();
                                    const uint32_t bw[8] = {bq[2 * c].x, bq[2 * c].y, bq[2 * c].z, bq[2 * c].w,
                                                            bq[2 * c + 1].x, bq[2 * c + 1].y, bq[2 * c + 1].z, bq[2 * c + 1].w};
#pragma unroll
                                    for (int e = 0; e < 8; ++e) {
                                        acc = fmaf(__uint_as_float(v[2 * e]), __uint_as_float(bw[e] << 16), acc);
                                        acc = fmaf(__uint_as_float(v[2 * e + 1]), __uint_as_float(bw[e] & 0xFFFF0000u), acc);
                                    }
                                }
                            }
                            yt[t] = acc;
                        }
                    }
                }
            }
            if (!ok) failed = true;
            if (csize == 1) {
                if (ok && i < p.m)
#pragma unroll
                    for (int t = 0; t < NTOK; ++t) store_out(p.y, p.y_f32, (size_t)t * p.m + i, yt[t]);
            } else {
                // a CTA that gave up still arrives (with zeros), so the leader never waits in vain
                const uint32_t leader_bar = map_to_rank(bar_reduce, 0);
#pragma unroll
                for (int t = 0; t < NTOK; ++t)
                    st_async_cluster_f32(map_to_rank(red0 + ((rank * NTOK + t) * kTileRows + row_in_tile) * 4, 0), yt[t], leader_bar);
                if (rank == 0) {
                    if (!__all_sync(0xffffffffu, mbar_wait_cluster(bar_reduce, 0, status, 9))) failed = true;
                    else if (i < p.m) {
                        // all partials are read first (the loads overlap), then added in rank order
                        float v[NTOK][kClusterMax];
#pragma unroll
                        for (int t = 0; t < NTOK; ++t)
#pragma unroll
                            for (int rr = 0; rr < kClusterMax; ++rr)
                                v[t][rr] = rr < csize ? __uint_as_float(lds_u32(red0 + ((rr * NTOK + t) * kTileRows + row_in_tile) * 4)) : 0.0f;
#pragma unroll
                        for (int t = 0; t < NTOK; ++t) {
                            float a = 0.0f;
#pragma unroll
                            for (int rr = 0; rr < kClusterMax; ++rr) a += v[t][rr];
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

// One (code width, tokens, halves) instantiation: its launch attributes, how many clusters of each
// size the device can hold at once, and the launch itself.
template <int BITS, int NTOK, int H> struct DecodeVariant {
    static int prepare(int dev)
    {
        static bool done[kMaxDevices] = {};
        if (!done[dev]) {
            auto kernel = lords_decode_kernel<BITS, NTOK, H>;
            LORDS_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, DCfg<BITS, H>::SMEM));
            // cluster sizes above 8 are outside the portable range; they are used only where the
            // occupancy query below says such a cluster fits
            LORDS_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
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
        // programmatic dependent launch: this kernel may start while the previous kernel in the stream
        // drains; it touches only weights until its griddepcontrol.wait
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg = cudaLaunchConfig_t{};
        cfg.gridDim = dim3((unsigned)(clusters * cs));
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = DCfg<BITS, H>::SMEM;
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
            const cudaError_t e = cudaOccupancyMaxActiveClusters(&n, lords_decode_kernel<BITS, NTOK, H>, &cfg);
            if (e != cudaSuccess) (void)cudaGetLastError();
            cache[dev][cs] = (e == cudaSuccess && n >= 1) ? n : -1;
        }
        return cache[dev][cs] > 0 ? cache[dev][cs] : 0;
    }
    static int launch(const DecodeParams &k, int tiles, int cs, cudaStream_t stream)
    {
        cudaLaunchConfig_t cfg;
        cudaLaunchAttribute attr[2];
        fill(cfg, attr, cs, tiles, stream);
        LORDS_CUDA_TRY(cudaLaunchKernelEx(&cfg, lords_decode_kernel<BITS, NTOK, H>, k));
        return LORDS_OK;
    }
};

// Cluster size for `tiles` tiles of `ksteps` k-steps: the largest split that still lets every cluster
// be resident at once (one wave); 1 when there are more tiles than that.  `cost` receives a relative
// time estimate, k-steps per CTA x waves x the per-step weight of the tile height.
template <int BITS, int NTOK, int H> int choose_cluster(int dev, int tiles, int ksteps, int forced, double &cost)
{
    using V = DecodeVariant<BITS, NTOK, H>;
    int cs = 1;
    if (forced > 0) {
        cs = forced < kClusterMax ? forced : kClusterMax;
        if (cs > ksteps) cs = ksteps;
        while (cs > 1 && V::max_clusters(dev, cs) == 0) --cs;
    } else {
        for (int c = kClusterMax < ksteps ? kClusterMax : ksteps; c > 1; --c)
            if (V::max_clusters(dev, c) >= tiles) { cs = c; break; }
    }
    const int resident = V::max_clusters(dev, cs) > 0 ? V::max_clusters(dev, cs) : 1;
    const int waves = (tiles + resident - 1) / resident;
    const int steps = (ksteps + cs - 1) / cs;
    // a two-half step covers twice the rows in about 1.7 times the time of a one-half step, and every
    // launch pays a fixed prologue + reduction worth a few steps
    cost = (double)waves * ((double)steps * (H == 2 ? 1.7 : 1.0) + 2.0);
    return cs;
}

template <int BITS, int NTOK> int launch_bits_tok(DecodeParams &k, const Problem &p, const State &st, cudaStream_t stream)
{
    const int dev = device_slot(st), forced_cs = st.forced_splitk;
    const int qrow = DCfg<BITS, 1>::QROW;
    k.ksteps = (p.n + kStep - 1) / kStep;
    int rc = DecodeVariant<BITS, NTOK, 1>::prepare(dev);
    if (rc == LORDS_OK) rc = DecodeVariant<BITS, NTOK, 2>::prepare(dev);
    if (rc != LORDS_OK) return rc;
    const int tiles1 = (p.m + 127) / 128, tiles2 = (p.m + 255) / 256;
    if (tiles1 > 65535) return LORDS_ERR_UNSUPPORTED;
    double cost1 = 0, cost2 = 0;
    const int cs1 = choose_cluster<BITS, NTOK, 1>(dev, tiles1, k.ksteps, forced_cs, cost1);
    const int cs2 = choose_cluster<BITS, NTOK, 2>(dev, tiles2, k.ksteps, forced_cs, cost2);
    const bool two = cost2 < cost1;
    const uint64_t row_bytes = (uint64_t)p.n * BITS / 8;
    if (!make_map_2d(&k.tm_q, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, p.q, row_bytes, (uint64_t)p.m, (uint32_t)qrow,
                     two ? 256u : 128u, BITS == 4 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !make_map_2d(&k.tm_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p.A, (uint64_t)p.n, (uint64_t)p.r, 64, (uint32_t)k.r_pad,
                     CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_2d(&k.tm_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p.x, (uint64_t)p.n, (uint64_t)p.M, (uint32_t)kStep, (uint32_t)NTOK,
                     CU_TENSOR_MAP_SWIZZLE_NONE))
        return LORDS_ERR_CUDA;
    k.tiles = two ? tiles2 : tiles1;
    return two ? DecodeVariant<BITS, NTOK, 2>::launch(k, tiles2, cs2, stream)
               : DecodeVariant<BITS, NTOK, 1>::launch(k, tiles1, cs1, stream);
}

}  // namespace

// Rules of this path: M <= 2 with M * ceil16(r) <= 64; n a multiple of 32 (4-bit), 64 (2-bit) or 128
// (3-bit), which makes every TMA row pitch a multiple of 16 bytes.  Anything else: LORDS_ERR_UNSUPPORTED.
int launch_decode(const Problem &p, State &st, cudaStream_t stream)
{
    if (p.bits < 2 || p.bits > 4) return LORDS_ERR_UNSUPPORTED;
    if (p.M > 2) return LORDS_ERR_UNSUPPORTED;
    const int r_pad = (p.r + 15) / 16 * 16;
    if (p.M * r_pad > kNMax) return LORDS_ERR_UNSUPPORTED;
    if (p.n % (p.bits == 4 ? 32 : p.bits == 2 ? 64 : 128) != 0) return LORDS_ERR_UNSUPPORTED;

    DecodeParams k;
    k.x = p.x; k.B = p.B;
    for (int c = 0; c < 16; ++c) k.levels[c] = p.levels[c];
    k.M = p.M; k.m = p.m; k.n = p.n; k.r = p.r; k.r_pad = r_pad;
    k.y = p.y; k.y_f32 = p.y_f32;
    k.status = st.status_word;
    int rc;
    if (p.bits == 4) rc = p.M == 1 ? launch_bits_tok<4, 1>(k, p, st, stream) : launch_bits_tok<4, 2>(k, p, st, stream);
    else if (p.bits == 3) rc = p.M == 1 ? launch_bits_tok<3, 1>(k, p, st, stream) : launch_bits_tok<3, 2>(k, p, st, stream);
    else rc = p.M == 1 ? launch_bits_tok<2, 1>(k, p, st, stream) : launch_bits_tok<2, 2>(k, p, st, stream);
    if (rc != LORDS_OK) return rc;
    st.last_launches = 1;
    st.last_path = "decode";
    return LORDS_OK;
}

}  // namespace lords
