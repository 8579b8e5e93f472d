// Quantisation step of the alternating refinement (Alg. 1, step 2.1; Sec. 3.3): with B and A fixed,
//
//     Q_ij = argmin over the codes c of (S_ij * L[c] - W_ij)^2,      S = B A (Eq. 3),
//
// written out as packed codes in the library's layout.  The paper does not say which level wins a tie:
// the lowest code does.  S is rebuilt tile by tile on the tensor cores exactly as the forward kernels
// rebuild it (bf16 operands from shared memory, fp32 in TMEM, never stored in full).  The decision is
// taken in fp32 with S accumulated in fp32: for a strictly ascending level table by bisection over the
// midpoints between neighbouring levels (log2 of the level count products and comparisons per weight),
// for any other table by trying every level in turn (one fused multiply-add and a square per level).
//
// One CTA owns 128 rows of W and a range of 64-column steps.  Warp roles (6 warps):
//   0..3  search: thread t owns row t; per step it reads its 64 values of S from TMEM (two loads of
//         32), its 64 weights from global memory, tries the levels, packs the codes and stores them.
//   4     TMEM allocation and MMA issuer: S[128 x 64] = B_tile (128 x r) * A_tile (r x 64) into one of
//         two TMEM buffers, as soon as the factor tile has landed and the buffer has been read.
//   5     TMA producer of the factor tiles A[:, step].
// Every wait is bounded; on expiry the role records LORDS_ERR_TIMEOUT and leaves its loop.
//
// Shapes outside the tensor-core rules (r > 64, n not a multiple of 64) take a plain CUDA-core kernel.
#include <cuda.h>
#include <cuda_bf16.h>

#include "lords_internal.h"
#include "lords_ptx.cuh"
#include "lords_tc_common.cuh"

namespace lords {

namespace {

using namespace ptx;

constexpr int kRowsQ = 128;                    // rows of W per CTA = UMMA M
constexpr int kColsQ = 64;                     // columns per step
constexpr int kSearchWarps = 4;
constexpr int kIssuerWarpQ = kSearchWarps;     // 4
constexpr int kTmaWarpQ = kSearchWarps + 1;    // 5
constexpr int kThreadsQ = (kSearchWarps + 2) * 32;
constexpr int kSAQ = 4;                        // factor-tile ring depth
constexpr int kSDQ = 2;                        // S buffers in TMEM
constexpr uint32_t kTmemColsQ = 128;
constexpr int kRMaxQ = 64;                     // largest rank of the tensor-core path (one swizzle atom of K)
constexpr int kATileBytesQ = kRMaxQ * 128;
constexpr int kBTileBytesQ = kRowsQ * 128;
constexpr int kSmemQ = 1024 + kSAQ * kATileBytesQ + kBTileBytesQ + 256;

struct alignas(64) QuantParams {
    CUtensorMap tm_a;     // bf16 [r][n], box {64, r_pad}, 128-byte swizzle (ranks past r read as zero)
    const uint16_t *W;    // bf16 [m][n]
    const uint16_t *B;    // bf16 [m][r]
    uint8_t *Q;           // packed codes, row pitch n * bits / 8
    float levels[16];
    float mids[16];       // ascending table: mids[c] = (levels[c] + levels[c + 1]) / 2
    int bits, m, n, r, r_pad;
    int steps;            // 64-column steps per row (n / 64)
    int steps_per_cta;
    int *status;
};

// The code whose level is nearest to w / s: every level in turn, the first (lowest) code keeps a tie.
template <int LEVELS>
__device__ __forceinline__ uint32_t nearest_code(float s, float w, const float (&lv)[16])
{
    uint32_t best = 0;
    const float d0 = fmaf(s, lv[0], -w);
    float e_best = d0 * d0;
#pragma unroll
    for (int c = 1; c < LEVELS; ++c) {
        const float d = fmaf(s, lv[c], -w);
        const float e = d * d;
        if (e < e_best) { e_best = e; best = (uint32_t)c; }
    }
    return best;
}

// The same for a strictly ascending table, by bisection over the midpoints between neighbouring levels:
// (s v - w)^2 = s^2 (v - w/s)^2, so the nearest level to t = w / s wins whatever the sign of s, and
// t > mid  <=>  b > a mid  with a = |s|, b = w sign(s).  The code is the number of midpoints below t; a
// weight exactly on a midpoint keeps the lower code, and s = 0 (every level equally good) gives code 0.
// The thresholds of the later steps are picked by selects on the earlier outcomes: log2(LEVELS)
// products and comparisons instead of LEVELS.
template <int LEVELS>
__device__ __forceinline__ uint32_t nearest_code_sorted(float s, float w, const float (&md)[16])
{
    const float a = fabsf(s);
    float b = s < 0.0f ? -w : w;
    b = a == 0.0f ? -INFINITY : b;
    if constexpr (LEVELS == 16) {
        const bool p3 = b > a * md[7];
        const bool p2 = b > a * (p3 ? md[11] : md[3]);
        const float m1 = p3 ? (p2 ? md[13] : md[9]) : (p2 ? md[5] : md[1]);
        const bool p1 = b > a * m1;
        const float m0hi = p2 ? (p1 ? md[14] : md[12]) : (p1 ? md[10] : md[8]);
        const float m0lo = p2 ? (p1 ? md[6] : md[4]) : (p1 ? md[2] : md[0]);
        const bool p0 = b > a * (p3 ? m0hi : m0lo);
        return ((uint32_t)p3 << 3) | ((uint32_t)p2 << 2) | ((uint32_t)p1 << 1) | (uint32_t)p0;
    } else if constexpr (LEVELS == 8) {
        const bool p2 = b > a * md[3];
        const bool p1 = b > a * (p2 ? md[5] : md[1]);
        const float m0 = p2 ? (p1 ? md[6] : md[4]) : (p1 ? md[2] : md[0]);
        const bool p0 = b > a * m0;
        return ((uint32_t)p2 << 2) | ((uint32_t)p1 << 1) | (uint32_t)p0;
    } else {
        const bool p1 = b > a * md[1];
        const bool p0 = b > a * (p1 ? md[2] : md[0]);
        return ((uint32_t)p1 << 1) | (uint32_t)p0;
    }
}

// 32 codes of one row -> packed bytes at `dst` (the row's byte offset of these 32 columns).
template <int BITS>
__device__ __forceinline__ void store_codes(uint8_t *dst, const uint32_t (&c)[32])
{
    if constexpr (BITS == 4) {
        uint32_t w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            uint32_t v = 0;
#pragma unroll
            for (int q = 0; q < 8; ++q) v |= c[8 * k + q] << (4 * q);
            w[k] = v;
        }
        *reinterpret_cast<uint4 *>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
    } else if constexpr (BITS == 3) {
        // a 96-bit little-endian integer, code j at bit 3j: codes 0..20 and the low bit of code 21 fill the
        // first 64 bits, the rest of code 21 and codes 22..31 the last 32
        unsigned long long a = 0;
#pragma unroll
        for (int j = 0; j < 21; ++j) a |= (unsigned long long)c[j] << (3 * j);
        a |= (unsigned long long)(c[21] & 1u) << 63;
        uint32_t hi = c[21] >> 1;
#pragma unroll
        for (int j = 22; j < 32; ++j) hi |= c[j] << (3 * j - 64);
        uint32_t *d = reinterpret_cast<uint32_t *>(dst);
        d[0] = (uint32_t)a;
        d[1] = (uint32_t)(a >> 32);
        d[2] = hi;
    } else {
        uint32_t w[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            uint32_t v = 0;
#pragma unroll
            for (int q = 0; q < 16; ++q) v |= c[16 * k + q] << (2 * q);
            w[k] = v;
        }
        *reinterpret_cast<uint2 *>(dst) = make_uint2(w[0], w[1]);
    }
}

template <int BITS, bool SORTED>
__global__ void __launch_bounds__(kThreadsQ, 3) lords_quantize_kernel(const __grid_constant__ QuantParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a0 = base;                                 // kSAQ factor tiles
    const uint32_t b_tile = a0 + kSAQ * kATileBytesQ;         // B[128 x 64 ranks] bf16, K-major, swizzled
    const uint32_t bars = b_tile + kBTileBytesQ;
    const uint32_t bar_a_full = bars, bar_a_free = bars + 8 * kSAQ;
    const uint32_t bar_s_full = bar_a_free + 8 * kSAQ, bar_s_free = bar_s_full + 8 * kSDQ;
    const uint32_t tmem_slot = bar_s_free + 8 * kSDQ;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row0 = (int)blockIdx.x * kRowsQ;
    const int st_a = (int)blockIdx.y * p.steps_per_cta;
    const int st_b = st_a + p.steps_per_cta < p.steps ? st_a + p.steps_per_cta : p.steps;
    const int total = st_b - st_a;
    const int *status = p.status;
    bool failed = false;

    if (tid == 0) {
        for (int b = 0; b < kSAQ; ++b) { mbar_init(bar_a_full + 8 * b, 1); mbar_init(bar_a_free + 8 * b, 1); }
        for (int b = 0; b < kSDQ; ++b) { mbar_init(bar_s_full + 8 * b, 1); mbar_init(bar_s_free + 8 * b, kSearchWarps); }
        fence_mbar_init();
    }
    if (warp == kIssuerWarpQ) {
        tmem_alloc(tmem_slot, kTmemColsQ);
        tmem_relinquish();
    } else if (warp < kSearchWarps) {
        // B tile: row rr = tid, 64 ranks (zero padded) bf16, K-major, 128-byte swizzle
        const int rr = tid, i = row0 + rr;
#pragma unroll
        for (int chunk = 0; chunk < 8; ++chunk) {
            uint32_t w4[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int k = chunk * 8 + e * 2;
                const uint32_t lo = (i < p.m && k < p.r) ? p.B[(size_t)i * p.r + k] : 0u;
                const uint32_t hi = (i < p.m && k + 1 < p.r) ? p.B[(size_t)i * p.r + k + 1] : 0u;
                w4[e] = lo | (hi << 16);
            }
            sts_v4(b_tile + (rr >> 3) * 1024 + (rr & 7) * 128 + ((chunk ^ (rr & 7)) * 16), make_uint4(w4[0], w4[1], w4[2], w4[3]));
        }
        fence_proxy_async_smem();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();

    if (warp == kTmaWarpQ) {
        if (lane == 0) {
            tma_prefetch_desc(&p.tm_a);
            const uint32_t tx = (uint32_t)(p.r_pad * 128);
            for (int it = 0; it < total; ++it) {
                const int sa = it % kSAQ;
                if (it >= kSAQ && !mbar_wait(bar_a_free + 8 * sa, (uint32_t)((it / kSAQ - 1) & 1), status, 31)) { failed = true; break; }
                const uint32_t bar = bar_a_full + 8 * sa;
                mbar_expect_tx(bar, tx);
                tma_load_2d(a0 + sa * kATileBytesQ, &p.tm_a, (st_a + it) * kColsQ, 0, bar);
            }
        }
    } else if (warp == kIssuerWarpQ) {
        uint32_t tmem_base;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
        constexpr uint32_t idesc = umma_idesc_f16(1, 0, 1, kRowsQ, kColsQ);     // bf16, B operand MN-major, N = 64
        const uint32_t desc_hi = (uint32_t)(umma_desc_sw128(0, 1024, 16) >> 32);
        const uint32_t lbo_lo = (uint32_t)umma_desc_sw128(0, 1024, 16);
        const uint32_t b_lo = lbo_lo | ((b_tile & 0x3FFFFu) >> 4);
        const uint32_t a_lo0 = lbo_lo | ((a0 & 0x3FFFFu) >> 4);
        const int ksteps = p.r_pad / 16;
        for (int it = 0; it < total; ++it) {
            const int sa = it % kSAQ, sd = it % kSDQ;
            if (!mbar_wait(bar_a_full + 8 * sa, (uint32_t)((it / kSAQ) & 1), status, 32)) { failed = true; break; }
            if (it >= kSDQ && !mbar_wait(bar_s_free + 8 * sd, (uint32_t)((it / kSDQ - 1) & 1), status, 33)) { failed = true; break; }
            tc_fence_after_sync();
            if (lane == 0) {
                const uint32_t a_lo = a_lo0 + (uint32_t)(sa * (kATileBytesQ >> 4));
                for (int k = 0; k < ksteps; ++k)
                    umma_f16_ss(tmem_base + (uint32_t)(sd * kColsQ), umma_desc_pack(b_lo + k * 2, desc_hi),
                                umma_desc_pack(a_lo + k * 128, desc_hi), idesc, k > 0);
                umma_commit(bar_s_full + 8 * sd);
                umma_commit(bar_a_free + 8 * sa);
            }
            __syncwarp();
        }
        // no commit is still on its way to a barrier when the CTA ends
        if (lane == 0 && !failed && total > 0) {
            const int last = total - 1;
            if (!mbar_wait(bar_a_free + 8 * (last % kSAQ), (uint32_t)((last / kSAQ) & 1), status, 34)) failed = true;
        }
    } else {
        const int i = row0 + tid;
        uint32_t tmem_base;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
        const uint32_t lane_addr = tmem_base + ((uint32_t)(warp * 32) << 16);
        float lv[16];
#pragma unroll
        for (int c = 0; c < 16; ++c) lv[c] = SORTED ? p.mids[c] : p.levels[c];
        const size_t qpitch = (size_t)p.n * BITS / 8;
        // the row's 32 weights of a half step are requested one half step ahead, so that their way
        // from HBM overlaps the search of the half step before
        uint4 wv[4], wn[4];
        auto load_w = [&](uint4 (&dst)[4], int it, int h) {
            if (i < p.m && it < total) {
                const uint4 *wp = reinterpret_cast<const uint4 *>(p.W + (size_t)i * p.n + (size_t)(st_a + it) * kColsQ + h * 32);
#pragma unroll
                for (int v = 0; v < 4; ++v) dst[v] = __ldg(wp + v);
            }
        };
        load_w(wv, 0, 0);
        for (int it = 0; it < total; ++it) {
            const int sd = it % kSDQ;
            const int col0 = (st_a + it) * kColsQ;
            if (!__all_sync(0xffffffffu, mbar_wait(bar_s_full + 8 * sd, (uint32_t)((it / kSDQ) & 1), status, 35))) { failed = true; break; }
            tc_fence_after_sync();
#pragma unroll 1
            for (int h = 0; h < 2; ++h) {
                uint32_t s[32];
                tmem_ld_32x32(lane_addr + (uint32_t)(sd * kColsQ + h * 32), s);
                load_w(wn, h == 0 ? it : it + 1, h == 0 ? 1 : 0);
                tmem_wait_ld();
                if (h == 1) {
                    // S is in registers: the buffer may be refilled
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_s_free + 8 * sd);
                }
                if (i < p.m) {
                    uint32_t codes[32];
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        const uint32_t ww[4] = {wv[v].x, wv[v].y, wv[v].z, wv[v].w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int c = v * 8 + e * 2;
                            const float w0 = __uint_as_float(ww[e] << 16), w1 = __uint_as_float(ww[e] & 0xFFFF0000u);
                            if constexpr (SORTED) {
                                codes[c] = nearest_code_sorted<(1 << BITS)>(__uint_as_float(s[c]), w0, lv);
                                codes[c + 1] = nearest_code_sorted<(1 << BITS)>(__uint_as_float(s[c + 1]), w1, lv);
                            } else {
                                codes[c] = nearest_code<(1 << BITS)>(__uint_as_float(s[c]), w0, lv);
                                codes[c + 1] = nearest_code<(1 << BITS)>(__uint_as_float(s[c + 1]), w1, lv);
                            }
                        }
                    }
                    store_codes<BITS>(p.Q + (size_t)i * qpitch + (size_t)(col0 + h * 32) * BITS / 8, codes);
                }
#pragma unroll
                for (int v = 0; v < 4; ++v) wv[v] = wn[v];
            }
        }
    }

    if (failed) atomicExch(p.status, LORDS_ERR_TIMEOUT);
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kIssuerWarpQ) {
        tc_fence_after_sync();
        uint32_t tmem_base;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
        tmem_dealloc(tmem_base, kTmemColsQ);
    }
}

// Plain CUDA-core version for any shape: a thread owns one row and one pack group of 32 columns (or what
// is left of the row), S by a loop over the ranks in fp32, the same level search.
template <int BITS>
__global__ void lords_quantize_simt_kernel(const uint16_t *__restrict__ W, const uint16_t *__restrict__ B,
                                           const uint16_t *__restrict__ A, uint8_t *__restrict__ Q, int m, int n, int r,
                                           const float *__restrict__ levels_dev)
{
    constexpr int LEVELS = 1 << BITS;
    constexpr int G = BITS == 3 ? 32 : (BITS == 4 ? 2 : 4);        // codes per whole number of bytes
    float lv[16];
#pragma unroll
    for (int c = 0; c < 16; ++c) lv[c] = c < LEVELS ? levels_dev[c] : 0.0f;
    const long long groups_per_row = n / G;
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= (long long)m * groups_per_row) return;
    const int i = (int)(gid / groups_per_row);
    const int j0 = (int)(gid % groups_per_row) * G;
    unsigned long long lo = 0;
    uint32_t hi = 0;
    for (int g = 0; g < G; ++g) {
        const int j = j0 + g;
        float s = 0.0f;
        for (int k = 0; k < r; ++k)
            s = fmaf(__uint_as_float((uint32_t)B[(size_t)i * r + k] << 16), __uint_as_float((uint32_t)A[(size_t)k * n + j] << 16), s);
        const uint32_t c = nearest_code<LEVELS>(s, __uint_as_float((uint32_t)W[(size_t)i * n + j] << 16), lv);
        const int bit = g * BITS;
        if (bit < 64) lo |= (unsigned long long)c << bit;
        if (bit + BITS > 64) hi |= bit >= 64 ? c << (bit - 64) : c >> (64 - bit);
    }
    uint8_t *dst = Q + (size_t)i * ((size_t)n * BITS / 8) + (size_t)j0 * BITS / 8;
    constexpr int BYTES = G * BITS / 8;
#pragma unroll
    for (int b = 0; b < BYTES; ++b) dst[b] = b < 8 ? (uint8_t)(lo >> (8 * b)) : (uint8_t)(hi >> (8 * (b - 8)));
}

template <int BITS, bool SORTED> int launch_quantize_tc(QuantParams &k, const State &st, cudaStream_t stream)
{
    static bool done[kMaxDevices] = {};
    const int dev = device_slot(st);
    if (!done[dev]) {
        LORDS_CUDA_TRY(cudaFuncSetAttribute(lords_quantize_kernel<BITS, SORTED>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemQ));
        done[dev] = true;
    }
    const int row_tiles = (k.m + kRowsQ - 1) / kRowsQ;
    // column ranges: about two CTAs per SM in all, at least four steps each
    int splits = (6 * st.sm_count + row_tiles - 1) / row_tiles;
    if (splits > k.steps / 4) splits = k.steps / 4;
    if (splits < 1) splits = 1;
    if (splits > 65535) splits = 65535;
    k.steps_per_cta = (k.steps + splits - 1) / splits;
    splits = (k.steps + k.steps_per_cta - 1) / k.steps_per_cta;
    lords_quantize_kernel<BITS, SORTED><<<dim3((unsigned)row_tiles, (unsigned)splits), kThreadsQ, kSmemQ, stream>>>(k);
    LORDS_CUDA_TRY(cudaGetLastError());
    return LORDS_OK;
}

}  // namespace

int launch_quantize(const void *W, const void *B, const void *A, const float *levels, int bits, int m, int n, int r,
                    uint8_t *Q, State &st, cudaStream_t stream)
{
    const bool tc = r <= kRMaxQ && n % kColsQ == 0;      // the row tiles are the grid's x dimension: any int fits
    if (tc && st.forced_path != 1) {
        QuantParams k;
        k.W = static_cast<const uint16_t *>(W); k.B = static_cast<const uint16_t *>(B); k.Q = Q;
        for (int c = 0; c < 16; ++c) k.levels[c] = c < (1 << bits) ? levels[c] : 0.0f;
        // a strictly ascending table (every NormalFloat table is) is searched by bisection over its
        // midpoints, any other table level by level
        bool sorted = true;
        for (int c = 0; c + 1 < (1 << bits); ++c) sorted = sorted && levels[c] < levels[c + 1];
        for (int c = 0; c < 16; ++c) k.mids[c] = (sorted && c + 1 < (1 << bits)) ? 0.5f * (levels[c] + levels[c + 1]) : 0.0f;
        k.bits = bits; k.m = m; k.n = n; k.r = r; k.r_pad = (r + 15) / 16 * 16;
        k.steps = n / kColsQ;
        k.status = st.status_word;
        if (!make_map_2d(&k.tm_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, A, (uint64_t)n, (uint64_t)r, 64, (uint32_t)k.r_pad,
                         CU_TENSOR_MAP_SWIZZLE_128B))
            return LORDS_ERR_CUDA;
        const int rc = sorted ? (bits == 4 ? launch_quantize_tc<4, true>(k, st, stream)
                                           : bits == 3 ? launch_quantize_tc<3, true>(k, st, stream) : launch_quantize_tc<2, true>(k, st, stream))
                              : (bits == 4 ? launch_quantize_tc<4, false>(k, st, stream)
                                           : bits == 3 ? launch_quantize_tc<3, false>(k, st, stream) : launch_quantize_tc<2, false>(k, st, stream));
        if (rc != LORDS_OK) return rc;
        st.last_launches = 1;
        st.last_path = "quantize";
        return LORDS_OK;
    }
    // CUDA-core version: the level table goes through the workspace (stream-ordered copy)
    if (st.workspace_bytes < 64) return LORDS_ERR_WORKSPACE;
    float *lv_dev = reinterpret_cast<float *>(st.workspace);
    LORDS_CUDA_TRY(cudaMemcpyAsync(lv_dev, levels, sizeof(float) * (size_t)(1 << bits), cudaMemcpyHostToDevice, stream));
    const int G = bits == 3 ? 32 : (bits == 4 ? 2 : 4);
    const long long work = (long long)m * (n / G);
    const unsigned blocks = (unsigned)((work + 127) / 128);
    const uint16_t *w16 = static_cast<const uint16_t *>(W), *b16 = static_cast<const uint16_t *>(B), *a16 = static_cast<const uint16_t *>(A);
    if (bits == 4) lords_quantize_simt_kernel<4><<<blocks, 128, 0, stream>>>(w16, b16, a16, Q, m, n, r, lv_dev);
    else if (bits == 3) lords_quantize_simt_kernel<3><<<blocks, 128, 0, stream>>>(w16, b16, a16, Q, m, n, r, lv_dev);
    else lords_quantize_simt_kernel<2><<<blocks, 128, 0, stream>>>(w16, b16, a16, Q, m, n, r, lv_dev);
    LORDS_CUDA_TRY(cudaGetLastError());
    st.last_launches = 1;
    st.last_path = "quantize_simt";
    return LORDS_OK;
}

}  // namespace lords
