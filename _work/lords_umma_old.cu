// Tensor-core path (sm_100a): TMA-staged operands, tcgen05.mma with accumulators in TMEM.
//
// One CTA owns a 128-row tile of W^ (out-features), a tile of BN tokens and a range of
// 64-column k-blocks (split-K over the in-feature axis).  Per k-block:
//   1. the TMA warp loads the packed code tile Q[128 x 64] (4-bit: 32 B per row), the factor
//      tile A[r x 64] (bf16) and the activation tile x16[BN x 64] (fp16) into a shared-memory ring;
//   2. the MMA thread issues the scale MMA  S = B_tile (128 x r) * A_tile (r x 64)  (Eq. 3,
//      bf16 operands, fp32 accumulator in TMEM);
//   3. eight dequant warps read S from TMEM, look up the levels of their codes, form
//      W^ = L[Q] (.) S as fp16 and store it as the 128-byte-swizzled K-major A operand;
//   4. the MMA thread issues  D[128 x BN] += W^_tile * x_tile^T  (fp16 operands, fp32 in TMEM).
// Epilogue: D -> registers -> y (bf16 RNE or fp32), or -> split-K scratch, where the last CTA
// of a tile to arrive adds the partials in split order (deterministic) and stores y.
//
// Every mbarrier wait is bounded; on expiry the kernel records LORDS_ERR_TIMEOUT, all roles
// drain, TMEM is released and the kernel returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "lords_internal.h"
#include "lords_ptx.cuh"

namespace lords {

namespace {

using namespace ptx;

constexpr int BM = 128;            // W^ rows per CTA = UMMA M
constexpr int BK = 64;             // in-feature columns per k-block (one swizzle row of fp16)
constexpr int kRMaxUmma = 64;      // largest rank this path takes (one swizzle atom of K)
constexpr int kDequantWarps = 8;
constexpr int kDequantThreads = kDequantWarps * 32;
constexpr int kTmaWarp = kDequantWarps;
constexpr int kMmaWarp = kDequantWarps + 1;
constexpr int kThreads = (kDequantWarps + 2) * 32;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kSCol = 256;    // S buffers live at TMEM columns 256 and 320
constexpr int kATileBytes = kRMaxUmma * 128;
constexpr int kQTileBytes = BM * 32;
constexpr int kWTileBytes = BM * 128;
constexpr int kLutBytes = 256 * 32 * 4;

template <int BN> struct Cfg {
    static constexpr int kStages = BN >= 256 ? 3 : 4;
    static constexpr int kXTileBytes = BN * 128;
    static constexpr int kStageBytes = kXTileBytes + kATileBytes + kQTileBytes;
    static constexpr int kSmemBytes = kStages * kStageBytes + 2 * kWTileBytes + kWTileBytes /*B tile*/ +
                                      kLutBytes + 256 /*barriers*/ + 1024 /*alignment slack*/;
};

struct alignas(64) UmmaParams {
    CUtensorMap tm_x;     // fp16 [M][n], box {64, BN}
    CUtensorMap tm_a;     // bf16 [r][n], box {64, r_pad}
    CUtensorMap tm_q;     // u8 [m][n/2], box {32, 128}
    const uint16_t *B;    // bf16 [m][r]
    float levels[16];
    int M, m, n, r, r_pad;
    int kblocks;          // ceil(n / 64)
    int splits, kb_per_split;
    int tok_tiles;
    float *partial;       // [splits][M][m]
    int *counters;        // one per (row tile, token tile), zero between calls
    void *y;
    int y_f32;
    int *status;
#ifdef LORDS_TRACE
    long long *trace;     // [3 roles][64 iterations][8 events] clock64 stamps of CTA 0 (debug builds only)
#endif
};

#ifdef LORDS_TRACE
#define LORDS_STAMP(role, it, ev)                                                        \
    do {                                                                                 \
        if (blockIdx.x == 0 && (it) < 64) p.trace[((role) * 64 + (it)) * 8 + (ev)] = clock64(); \
    } while (0)
#else
#define LORDS_STAMP(role, it, ev) do { } while (0)
#endif

__device__ __forceinline__ void store_out(void *y, int y_f32, size_t idx, float v)
{
    if (y_f32) static_cast<float *>(y)[idx] = v;
    else static_cast<__nv_bfloat16 *>(y)[idx] = __float2bfloat16_rn(v);
}

__device__ __forceinline__ void named_bar_sync(int id, int count)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

template <int BN>
__global__ void __launch_bounds__(kThreads, 1) lords_umma_kernel(const __grid_constant__ UmmaParams p)
{
    using C = Cfg<BN>;
    constexpr int STAGES = C::kStages;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (base - raw);

    // carve-up (all tile bases are multiples of 1024 bytes)
    const uint32_t x_tile0 = base;
    const uint32_t a_tile0 = x_tile0 + STAGES * C::kXTileBytes;
    const uint32_t q_tile0 = a_tile0 + STAGES * kATileBytes;
    const uint32_t w_tile0 = q_tile0 + STAGES * kQTileBytes;
    const uint32_t b_tile = w_tile0 + 2 * kWTileBytes;
    const uint32_t lut_addr = b_tile + kWTileBytes;
    const uint32_t bars = lut_addr + kLutBytes;
    const uint32_t bar_tma_full = bars;                 // STAGES
    const uint32_t bar_tma_empty = bars + 8 * 4;        // STAGES
    const uint32_t bar_s_full = bars + 8 * 8;           // 2
    const uint32_t bar_w_full = bars + 8 * 10;          // 2
    const uint32_t bar_w_empty = bars + 8 * 12;         // 2
    const uint32_t bar_acc_full = bars + 8 * 14;        // 1
    const uint32_t tmem_slot = bars + 8 * 16;           // u32
    uint8_t *sm_q = sm + (q_tile0 - base);
    uint8_t *sm_w = sm + (w_tile0 - base);
    uint8_t *sm_b = sm + (b_tile - base);
    __half2 *sm_lut = reinterpret_cast<__half2 *>(sm + (lut_addr - base));
    volatile uint32_t *sm_tmem = reinterpret_cast<volatile uint32_t *>(sm + (tmem_slot - base));
    __shared__ float s_levels[16];
    __shared__ int s_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // work assignment
    const int tiles_per_split = (int)gridDim.x / p.splits;
    const int split = (int)blockIdx.x / tiles_per_split;
    const int tile = (int)blockIdx.x - split * tiles_per_split;
    const int row_tile = tile / p.tok_tiles;
    const int tok_tile = tile - row_tile * p.tok_tiles;
    const int row0 = row_tile * BM;
    const int tok0 = tok_tile * BN;
    const int kb0 = split * p.kb_per_split;
    const int nkb = min(p.kb_per_split, p.kblocks - kb0);

    if (tid < 16) s_levels[tid] = p.levels[tid];
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_tma_full + 8 * s, 1);
            mbar_init(bar_tma_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_s_full + 8 * b, 1);
            mbar_init(bar_w_full + 8 * b, kDequantThreads);
            mbar_init(bar_w_empty + 8 * b, 1);
        }
        mbar_init(bar_acc_full, 1);
        fence_mbar_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    if (warp == kTmaWarp && lane == 0) {
        tma_prefetch_desc(&p.tm_x);
        tma_prefetch_desc(&p.tm_a);
        tma_prefetch_desc(&p.tm_q);
    }
    __syncthreads();   // s_levels visible

    if (warp < kDequantWarps) {
        // level-pair table: entry e = (L[e & 15], L[e >> 4]) as fp16x2, one private copy per lane
        // (word e*32 + lane sits in bank `lane`: lookups never conflict)
        for (int e0 = 0; e0 < 256; e0 += kDequantWarps) {
            const int e = e0 + warp;
            sm_lut[e * 32 + lane] = __floats2half2_rn(s_levels[e & 15], s_levels[e >> 4]);
        }
        // B tile: 128 rows x 64 ranks (zero padded) bf16, K-major, 128-byte swizzle
        {
            const int rr = tid >> 1, half = tid & 1;
            const int i = row0 + rr;
            for (int c = 0; c < 4; ++c) {
                const int chunk = half * 4 + c;
                uint32_t w4[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int k = chunk * 8 + e * 2;
                    uint32_t lo = (i < p.m && k < p.r) ? p.B[(size_t)i * p.r + k] : 0u;
                    uint32_t hi = (i < p.m && k + 1 < p.r) ? p.B[(size_t)i * p.r + k + 1] : 0u;
                    w4[e] = lo | (hi << 16);
                }
                uint8_t *dst = sm_b + (rr >> 3) * 1024 + (rr & 7) * 128 + ((chunk ^ (rr & 7)) * 16);
                *reinterpret_cast<uint4 *>(dst) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
            }
        }
        fence_proxy_async_smem();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *sm_tmem;

    bool failed = false;

    if (warp == kTmaWarp) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint32_t stage_tx = (uint32_t)(C::kXTileBytes + p.r_pad * 128 + kQTileBytes);
            for (int it = 0; it < nkb; ++it) {
                const int st = it % STAGES;
                if (it >= STAGES && !mbar_wait(bar_tma_empty + 8 * st, (uint32_t)((it / STAGES - 1) & 1))) {
                    failed = true;
                    break;
                }
                LORDS_STAMP(2, it, 0);
                const int j0 = (kb0 + it) * BK;
                const uint32_t bar = bar_tma_full + 8 * st;
                mbar_expect_tx(bar, stage_tx);
                tma_load_2d(q_tile0 + st * kQTileBytes, &p.tm_q, j0 / 2, row0, bar);
                tma_load_2d(a_tile0 + st * kATileBytes, &p.tm_a, j0, 0, bar);
                tma_load_2d(x_tile0 + st * C::kXTileBytes, &p.tm_x, j0, tok0, bar);
                LORDS_STAMP(2, it, 1);
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_s = umma_idesc_f16(1, 0, 1, BM, 64);     // bf16, B operand MN-major
            constexpr uint32_t idesc_m = umma_idesc_f16(0, 0, 0, BM, BN);     // fp16, both K-major
            const int ksteps = p.r_pad / 16;
            auto issue_scale = [&](int it) -> bool {
                const int st = it % STAGES, buf = it & 1;
                if (!mbar_wait(bar_tma_full + 8 * st, (uint32_t)((it / STAGES) & 1))) return false;
                tc_fence_after_sync();
                for (int k = 0; k < ksteps; ++k) {
                    const uint64_t ad = umma_desc_sw128(b_tile + k * 32, 1024, 16);
                    const uint64_t bd = umma_desc_sw128(a_tile0 + st * kATileBytes + k * 2048, 1024, 16);
                    umma_f16_ss(tmem_base + kSCol + buf * 64, ad, bd, idesc_s, k > 0);
                }
                umma_commit(bar_s_full + 8 * buf);
                return true;
            };
            bool ok = nkb > 0 ? issue_scale(0) : true;
            if (ok && nkb > 1) ok = issue_scale(1);
            for (int it = 0; ok && it < nkb; ++it) {
                const int st = it % STAGES, buf = it & 1;
                LORDS_STAMP(0, it, 0);
                if (!mbar_wait(bar_w_full + 8 * buf, (uint32_t)((it >> 1) & 1))) { ok = false; break; }
                tc_fence_after_sync();
                LORDS_STAMP(0, it, 1);
#pragma unroll
                for (int k = 0; k < BK / 16; ++k) {
                    const uint64_t ad = umma_desc_sw128(w_tile0 + buf * kWTileBytes + k * 32, 1024, 16);
                    const uint64_t bd = umma_desc_sw128(x_tile0 + st * C::kXTileBytes + k * 32, 1024, 16);
                    umma_f16_ss(tmem_base, ad, bd, idesc_m, (it > 0 || k > 0) ? 1u : 0u);
                }
                umma_commit(bar_tma_empty + 8 * st);
                umma_commit(bar_w_empty + 8 * buf);
                LORDS_STAMP(0, it, 2);
                if (it + 2 < nkb) ok = issue_scale(it + 2);
                LORDS_STAMP(0, it, 3);
            }
            umma_commit(bar_acc_full);
            failed = !ok;
        }
    } else {
        // ------------------------------------------------------------------ dequant warps
        const int quad = warp & 3, half = warp >> 2;
        const int row = quad * 32 + lane;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        const __half2 *lut = sm_lut + lane;
        for (int it = 0; it < nkb; ++it) {
            const int st = it % STAGES, buf = it & 1;
            if (tid == 0) LORDS_STAMP(1, it, 0);
            if (!__all_sync(0xffffffffu, mbar_wait(bar_s_full + 8 * buf, (uint32_t)((it >> 1) & 1)))) { failed = true; break; }
            tc_fence_after_sync();
            if (tid == 0) LORDS_STAMP(1, it, 1);
            uint32_t s[32];
            tmem_ld_32x32(lane_addr + kSCol + buf * 64 + half * 32, s);
            if (!__all_sync(0xffffffffu, mbar_wait(bar_tma_full + 8 * st, (uint32_t)((it / STAGES) & 1)))) {
                tmem_wait_ld();
                failed = true;
                break;
            }
            const uint4 cw = *reinterpret_cast<const uint4 *>(sm_q + st * kQTileBytes + row * 32 + half * 16);
            tmem_wait_ld();
            if (tid == 0) LORDS_STAMP(1, it, 2);
            const uint32_t cwv[4] = {cw.x, cw.y, cw.z, cw.w};
            uint32_t out[16];
#pragma unroll
            for (int b = 0; b < 16; ++b) {
                const uint32_t byte = (cwv[b >> 2] >> (8 * (b & 3))) & 0xFFu;
                const __half2 lv = lut[byte * 32];
                const __half2 sv = __floats2half2_rn(__uint_as_float(s[2 * b]), __uint_as_float(s[2 * b + 1]));
                const __half2 wv = __hmul2(lv, sv);
                out[b] = *reinterpret_cast<const uint32_t *>(&wv);
            }
            if (it >= 2 && !__all_sync(0xffffffffu, mbar_wait(bar_w_empty + 8 * buf, (uint32_t)(((it >> 1) - 1) & 1)))) {
                failed = true;
                break;
            }
            if (tid == 0) LORDS_STAMP(1, it, 3);
            uint8_t *wrow = sm_w + buf * kWTileBytes + (row >> 3) * 1024 + (row & 7) * 128;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int chunk = (half * 4 + c) ^ (row & 7);
                *reinterpret_cast<uint4 *>(wrow + chunk * 16) =
                    make_uint4(out[4 * c], out[4 * c + 1], out[4 * c + 2], out[4 * c + 3]);
            }
            if (tid == 0) LORDS_STAMP(1, it, 4);
            fence_proxy_async_smem();
            tc_fence_before_sync();
            if (tid == 0) LORDS_STAMP(1, it, 5);
            mbar_arrive(bar_w_full + 8 * buf);
            if (tid == 0) LORDS_STAMP(1, it, 6);
        }

        // ------------------------------------------------------------------ epilogue
        if (!failed && !__all_sync(0xffffffffu, mbar_wait(bar_acc_full, 0))) failed = true;
        failed = __any_sync(0xffffffffu, failed);
        tc_fence_after_sync();
        if (!failed && nkb > 0) {
            const int i = row0 + row;
            constexpr int kColsPerHalf = BN >= 32 ? BN / 2 : BN;
            const bool active = BN >= 32 || half == 0;
            if (active) {
                for (int c0 = half * kColsPerHalf; c0 < (half + 1) * kColsPerHalf; c0 += 16) {
                    uint32_t v[16];
                    tmem_ld_32x16(lane_addr + c0, v);
                    tmem_wait_ld();
                    if (i < p.m) {
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const int t = tok0 + c0 + c;
                            if (t < p.M) {
                                const float f = __uint_as_float(v[c]);
                                if (p.splits > 1) p.partial[((size_t)split * p.M + t) * p.m + i] = f;
                                else store_out(p.y, p.y_f32, (size_t)t * p.m + i, f);
                            }
                        }
                    }
                }
            }
        }
        tc_fence_before_sync();

        if (p.splits > 1) {
            // last CTA of this (row tile, token tile) to arrive adds the partials in split order
            __threadfence();
            named_bar_sync(1, kDequantThreads);
            if (tid == 0) {
                const int prev = atomicAdd(p.counters + tile, 1);
                const int last = (prev == p.splits - 1);
                if (last) p.counters[tile] = 0;
                s_last = last;
            }
            named_bar_sync(1, kDequantThreads);
            if (s_last) {
                __threadfence();
                const int ntok = min(BN, p.M - tok0);
                const int rr = tid & (BM - 1);
                const int i = row0 + rr;
                if (i < p.m) {
                    for (int tt = tid >> 7; tt < ntok; tt += kDequantThreads / BM) {
                        const int t = tok0 + tt;
                        float acc = 0.0f;
                        for (int s = 0; s < p.splits; ++s) acc += __ldcg(p.partial + ((size_t)s * p.M + t) * p.m + i);
                        store_out(p.y, p.y_f32, (size_t)t * p.m + i, acc);
                    }
                }
            }
        }
    }

    if (failed) atomicExch(p.status, LORDS_ERR_TIMEOUT);
    __syncthreads();
    if (warp == kMmaWarp) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// x bf16 -> fp16 (exact for every bf16 value inside fp16's normal range), 8 elements per thread.
__global__ void lords_x_to_f16_kernel(const uint4 *__restrict__ x, uint4 *__restrict__ x16, size_t n_vec)
{
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

bool make_map_2d(CUtensorMap *map, CUtensorMapDataType dt, int elem_bytes, const void *ptr, uint64_t inner,
                 uint64_t outer, uint32_t box_inner, uint32_t box_outer, CUtensorMapSwizzle swz)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {inner * (uint64_t)elem_bytes};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    CUresult rc = fn(map, dt, 2, const_cast<void *>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS;
}

template <int BN> int launch_bn(const UmmaParams &k, int grid, cudaStream_t stream)
{
    static bool attr_set = false;
    if (!attr_set) {
        LORDS_CUDA_TRY(cudaFuncSetAttribute(lords_umma_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            Cfg<BN>::kSmemBytes));
        attr_set = true;
    }
    lords_umma_kernel<BN><<<grid, kThreads, Cfg<BN>::kSmemBytes, stream>>>(k);
    LORDS_CUDA_TRY(cudaGetLastError());
    return LORDS_OK;
}

}  // namespace

// Returns LORDS_ERR_UNSUPPORTED when the shape is outside this path's rules:
// 4-bit codes, n a multiple of 64, r <= 64, scratch large enough.
int launch_umma(const Problem &p, State &st, cudaStream_t stream)
{
    if (p.bits != 4 || p.n % 64 != 0 || p.r > kRMaxUmma) return LORDS_ERR_UNSUPPORTED;

    const int BN = p.M <= 16 ? 16 : p.M <= 32 ? 32 : p.M <= 64 ? 64 : p.M <= 128 ? 128 : 256;
    UmmaParams k;
    k.B = p.B;
    for (int c = 0; c < 16; ++c) k.levels[c] = p.levels[c];
    k.M = p.M; k.m = p.m; k.n = p.n; k.r = p.r;
    k.r_pad = (p.r + 15) / 16 * 16;
    k.kblocks = p.n / BK;
    k.tok_tiles = (p.M + BN - 1) / BN;
    const int row_tiles = (p.m + BM - 1) / BM;
    const long tiles = (long)row_tiles * k.tok_tiles;
    if (tiles > st.counter_slots) return LORDS_ERR_UNSUPPORTED;

    int splits = st.forced_splitk;
    if (splits <= 0) {
        splits = (int)(st.sm_count / tiles);                 // one wave: never more CTAs than SMs
        if (splits > k.kblocks / 4) splits = k.kblocks / 4;  // at least 4 k-blocks per CTA
        if (splits < 1) splits = 1;
    }
    if (splits > k.kblocks) splits = k.kblocks;
    k.kb_per_split = (k.kblocks + splits - 1) / splits;
    splits = (k.kblocks + k.kb_per_split - 1) / k.kb_per_split;
    k.splits = splits;

    // scratch: [ x as fp16 | split-K partials ]
    const size_t x16_bytes = ((size_t)p.M * p.n * 2 + 1023) & ~(size_t)1023;
    const size_t part_bytes = splits > 1 ? (size_t)splits * p.M * p.m * sizeof(float) : 0;
    if (x16_bytes + part_bytes > st.workspace_bytes) return LORDS_ERR_WORKSPACE;
    uint8_t *x16 = st.workspace;
    k.partial = reinterpret_cast<float *>(st.workspace + x16_bytes);
    k.counters = st.counters;
    k.y = p.y; k.y_f32 = p.y_f32;
    k.status = st.status_word;
#ifdef LORDS_TRACE
    k.trace = reinterpret_cast<long long *>(st.workspace + st.workspace_bytes - (size_t)3 * 64 * 8 * 8);
    LORDS_CUDA_TRY(cudaMemsetAsync(k.trace, 0, (size_t)3 * 64 * 8 * 8, stream));
#endif

    if (!make_map_2d(&k.tm_x, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, x16, (uint64_t)p.n, (uint64_t)p.M, 64, (uint32_t)BN,
                     CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_2d(&k.tm_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p.A, (uint64_t)p.n, (uint64_t)p.r, 64,
                     (uint32_t)k.r_pad, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_2d(&k.tm_q, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, p.q, (uint64_t)p.n / 2, (uint64_t)p.m, 32, BM,
                     CU_TENSOR_MAP_SWIZZLE_NONE))
        return LORDS_ERR_CUDA;

    const size_t n_vec = (size_t)p.M * p.n / 8;
    lords_x_to_f16_kernel<<<(unsigned)((n_vec + 255) / 256), 256, 0, stream>>>(
        reinterpret_cast<const uint4 *>(p.x), reinterpret_cast<uint4 *>(x16), n_vec);
    LORDS_CUDA_TRY(cudaGetLastError());

    const int grid = (int)(tiles * splits);
    int rc;
    switch (BN) {
        case 16: rc = launch_bn<16>(k, grid, stream); break;
        case 32: rc = launch_bn<32>(k, grid, stream); break;
        case 64: rc = launch_bn<64>(k, grid, stream); break;
        case 128: rc = launch_bn<128>(k, grid, stream); break;
        default: rc = launch_bn<256>(k, grid, stream); break;
    }
    if (rc != LORDS_OK) return rc;
    st.last_launches = 2;
    st.last_path = "umma";
    return LORDS_OK;
}

#ifdef LORDS_TRACE
// Debug builds only: copy CTA 0's clock stamps of the last tensor-core launch to the host.
extern "C" int lords_debug_read_trace(long long *out)
{
    State &st = state();
    if (!st.initialised) return LORDS_ERR_NOT_INIT;
    LORDS_CUDA_TRY(cudaDeviceSynchronize());
    LORDS_CUDA_TRY(cudaMemcpy(out, st.workspace + st.workspace_bytes - (size_t)3 * 64 * 8 * 8, (size_t)3 * 64 * 8 * 8,
                              cudaMemcpyDeviceToHost));
    return LORDS_OK;
}
#endif

}  // namespace lords
