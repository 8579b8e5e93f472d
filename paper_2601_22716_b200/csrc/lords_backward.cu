// Backward of the layer y = x W^T, W^ = L[Q] (.) (B A), with the codes fixed: the gradients that
// multiplicative fine-tuning of B and A needs (Sec. 3.4; the chain rule through S = BA is the one of
// Eq. 5).  With g = dL/dy (M x m):
//
//     dx = g W^                                   (M x n)
//     dS = (g^T x) (.) L[Q]                       (m x n, never stored: built tile by tile)
//     dB = dS A^T   (m x r),     dA = B^T dS      (r x n)
//
// dx is the forward operator of the transposed layer: W^T = L[Q^T] (.) (A^T B^T), so with a transposed
// copy of the packed codes (made once: the codes are frozen) and the transposed factors it runs on the
// forward kernels as they are.  This file holds what that needs -- the transposition of packed codes
// and of the two factors -- and the kernels for dB and dA.
//
// The same kernels give the straight-through gradients of quantisation-aware training (Sec. 3.3, Eq. 4-5):
// the tile of g^T x is dL/dW^ = dL/dW itself, and the factor of dL/dS is L[Q] - W (/) S instead of L[Q],
// with S = B A rebuilt per tile (by a scale MMA on the tensor schedule where the rank allows it).
//
// dB and dA: a tile of dS is formed by the product g^T x over the tokens, multiplied by the levels of
// the tile's codes, and folded with the matching column slice of A (for dB) and row slice of B (for
// dA); bf16 inputs are widened exactly, sums are fp32.  Three schedules:
//   tiles: one CTA per 64 x 64 tile of W, everything on the CUDA cores; it writes the tile's contributions to dB and dA into the library's
//          workspace, and a second kernel adds the contributions of a row (or column) of tiles in tile
//          order.  g^T x is formed once, and the grid fills the machine.  Taken when the workspace
//          holds the contributions (4 r (m n / 64 + n m / 64) bytes).
//   walk:  one CTA per 64 rows (dB) or 64 columns (dA) walks over the other dimension and keeps its
//          sums in registers.  No scratch memory, g^T x formed once per gradient.
//   tensor: the first schedule with the tile product g^T x on the tensor cores (tcgen05, bf16 operands
//          straight from g and x by TMA, fp32 accumulator in TMEM) and only the level multiply and
//          the two folds (register-blocked, operands from shared memory as 16-byte words) on the CUDA
//          cores.  Taken when the row pitches suit TMA (m, n multiples of 8).
// Either way every output element is summed in a fixed order without atomics: runs are bit-identical.
// Bound: fp32 ALU, m n M fused multiply-adds for the tile product (twice with the walk), or, with the
// tensor schedule, the 2 m n r multiply-adds of the folds.
#include <cuda.h>
#include <cuda_runtime.h>

#include <type_traits>

#include "lords_internal.h"
#include "lords_ptx.cuh"
#include "lords_tc_common.cuh"

namespace lords {

namespace {

using namespace ptx;

__device__ __forceinline__ float bf16f(uint16_t h) { return __uint_as_float((uint32_t)h << 16); }

// Code (i, j) of a packed row-major code matrix with `row_bytes` bytes per row.
__device__ __forceinline__ uint32_t read_code(const uint8_t *__restrict__ q, size_t row_bytes, int i, int j, int bits)
{
    const uint8_t *row = q + (size_t)i * row_bytes;
    const int bit = j * bits, byte = bit >> 3, sh = bit & 7;
    uint32_t v = row[byte];
    if (sh + bits > 8) v |= (uint32_t)row[byte + 1] << 8;
    return (v >> sh) & ((1u << bits) - 1u);
}

// ---- transposition of packed codes -----------------------------------------------------------------
// Thread (j, group): the codes Q[i0 .. i0 + 31][j] become 32 consecutive codes of row j of Q^T.
// Neighbouring threads take neighbouring j, so the reads of one row of Q are contiguous.
__global__ void lords_transpose_codes_kernel(const uint8_t *__restrict__ Q, uint8_t *__restrict__ Qt, int m, int n, int bits)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int i0 = blockIdx.y * 32;
    if (j >= n) return;
    const size_t row_bytes = (size_t)n * bits / 8, trow_bytes = (size_t)m * bits / 8;
    const int count = m - i0 < 32 ? m - i0 : 32;        // a multiple of the pack group, like m
    unsigned long long lo = 0;                          // up to 128 bits of packed codes
    unsigned long long hi = 0;
    for (int ii = 0; ii < count; ++ii) {
        const unsigned long long c = read_code(Q, row_bytes, i0 + ii, j, bits);
        const int bit = ii * bits;
        if (bit < 64) {
            lo |= c << bit;
            if (bit + bits > 64) hi |= c >> (64 - bit);
        } else {
            hi |= c << (bit - 64);
        }
    }
    uint8_t *dst = Qt + (size_t)j * trow_bytes + (size_t)i0 * bits / 8;
    const int bytes = count * bits / 8;
    for (int b = 0; b < bytes; ++b) dst[b] = (uint8_t)(b < 8 ? lo >> (8 * b) : hi >> (8 * (b - 8)));
}

// Two transpositions in one launch (the factors A and B of a layer): blocks [0, tiles0) take the first matrix,
// the others the second.
__global__ void lords_transpose_bf16_pair_kernel(const uint16_t *__restrict__ src0, uint16_t *__restrict__ dst0, int rows0, int cols0,
                                                 const uint16_t *__restrict__ src1, uint16_t *__restrict__ dst1, int rows1, int cols1,
                                                 int tiles0)
{
    __shared__ uint16_t tile[32][33];
    const bool first = (int)blockIdx.x < tiles0;
    const uint16_t *src = first ? src0 : src1;
    uint16_t *dst = first ? dst0 : dst1;
    const int rows = first ? rows0 : rows1, cols = first ? cols0 : cols1;
    const int t = first ? (int)blockIdx.x : (int)blockIdx.x - tiles0, tiles_x = (cols + 31) / 32;
    const int c0 = (t % tiles_x) * 32, r0 = (t / tiles_x) * 32;
    for (int k = threadIdx.y; k < 32; k += blockDim.y) {
        const int rr = r0 + k, cc = c0 + threadIdx.x;
        tile[k][threadIdx.x] = (rr < rows && cc < cols) ? src[(size_t)rr * cols + cc] : (uint16_t)0;
    }
    __syncthreads();
    for (int k = threadIdx.y; k < 32; k += blockDim.y) {
        const int cc = c0 + k, rr = r0 + threadIdx.x;
        if (cc < cols && rr < rows) dst[(size_t)cc * rows + rr] = tile[threadIdx.x][k];
    }
}

// ---- dB and dA -------------------------------------------------------------------------------------------
constexpr int kT = 64;          // tile edge (rows of W and columns of W per step)
constexpr int kTok = 16;        // tokens per shared-memory slice of the g^T x product
constexpr int kBwThreads = 256;
constexpr int kRMaxBw = 128;    // = LORDS_R_MAX

struct BwParams {
    const uint16_t *g;    // bf16 [M][m]
    const uint16_t *x;    // bf16 [M][n]
    const uint8_t *q;     // packed codes [m][n * bits / 8]
    const uint16_t *B;    // bf16 [m][r]
    const uint16_t *A;    // bf16 [r][n]
    float levels[16];
    int bits, M, m, n, r;
    float *dB;            // [m][r]
    float *dA;            // [r][n]
    // quantisation-aware training (Eq. 4-5), schedule "walk": the latent weight (null: fine-tuning with
    // the codes fixed) and where dL/dW goes (null: not asked for)
    const uint16_t *W;    // bf16 [m][n]
    float *dW;            // float [m][n]
};

// ROLE 0: dB for rows blockIdx.x * 64 ..; ROLE 1: dA for columns blockIdx.x * 64 ...
// With p.W set the factor of dL/dS is L[Q] - W (/) S (Eq. 5; S = B A rebuilt per tile in fp32, summed over
// the rank in ascending order; 0 where S is 0), and the launch with write_dW set also stores the tile of
// g^T x as dL/dW (Eq. 4).
template <int ROLE>
__global__ void __launch_bounds__(kBwThreads) lords_backward_factors_kernel(const BwParams p, const int write_dW)
{
    __shared__ __align__(16) float gs[kTok][kT];   // g[t][i0 + ..]
    __shared__ __align__(16) float xs[kTok][kT];   // x[t][j0 + ..]
    __shared__ float ds[kT][kT + 1];               // dS tile
    __shared__ uint16_t fs[kRMaxBw][kT + 2];       // ROLE 0: A[k][j0 + ..]; ROLE 1: B[i0 + ..][k] stored [k][i]
                                                   // (rows 33 words apart: neighbouring k fall into different banks)
    __shared__ float lv_s[16];                     // the level table (a per-thread index into the kernel parameters is replayed per distinct value)

    const int tid = threadIdx.x;
    if (tid < 16) lv_s[tid] = p.levels[tid];       // read after the first __syncthreads below
    const int ty = tid >> 4, tx = tid & 15;   // 16 x 16 threads, a 4 x 4 micro-tile each
    const int own0 = blockIdx.x * kT;         // first owned row (ROLE 0) or column (ROLE 1)
    const int walk_len = ROLE == 0 ? p.n : p.m;
    const size_t row_bytes = (size_t)p.n * p.bits / 8;

    // accumulators: output element e = tid + 256 * a of the owned [64][r] (ROLE 0: [i][k]) or [r][64]
    // (ROLE 1: [k][j]) block
    // (r rounded up to a multiple of 4, so that the block is a whole number of elements per thread)
    constexpr int kAccMax = kRMaxBw * kT / kBwThreads;     // 32
    float acc[kAccMax];
    const int r4 = (p.r + 3) & ~3;
    const int nacc4 = r4 * kT / kBwThreads;
#pragma unroll
    for (int a = 0; a < kAccMax; ++a) acc[a] = 0.0f;

    for (int w0 = 0; w0 < walk_len; w0 += kT) {
        const int i0 = ROLE == 0 ? own0 : w0, j0 = ROLE == 0 ? w0 : own0;
        // ---- tile of g^T x over all tokens
        float c[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) c[a][b] = 0.0f;
        for (int t0 = 0; t0 < p.M; t0 += kTok) {
            for (int e = tid; e < kTok * kT; e += kBwThreads) {
                const int t = t0 + e / kT, cidx = e % kT;
                gs[e / kT][cidx] = (t < p.M && i0 + cidx < p.m) ? bf16f(p.g[(size_t)t * p.m + i0 + cidx]) : 0.0f;
                xs[e / kT][cidx] = (t < p.M && j0 + cidx < p.n) ? bf16f(p.x[(size_t)t * p.n + j0 + cidx]) : 0.0f;
            }
            __syncthreads();
#pragma unroll
            for (int t = 0; t < kTok; ++t) {
                const float4 g4 = *reinterpret_cast<const float4 *>(&gs[t][ty * 4]);
                const float4 x4 = *reinterpret_cast<const float4 *>(&xs[t][tx * 4]);
                const float gv[4] = {g4.x, g4.y, g4.z, g4.w}, xv[4] = {x4.x, x4.y, x4.z, x4.w};
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int b = 0; b < 4; ++b) c[a][b] = fmaf(gv[a], xv[b], c[a][b]);
            }
            __syncthreads();
        }
        // ---- QAT: the tile of S = B A, by the same outer-product steps with the rank in place of the tokens
        float sc[4][4];
        if (p.W) {
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) sc[a][b] = 0.0f;
            for (int k0 = 0; k0 < p.r; k0 += kTok) {
                for (int e = tid; e < kTok * kT; e += kBwThreads) {
                    const int k = k0 + e / kT, cidx = e % kT;
                    gs[e / kT][cidx] = (k < p.r && i0 + cidx < p.m) ? bf16f(p.B[(size_t)(i0 + cidx) * p.r + k]) : 0.0f;
                    xs[e / kT][cidx] = (k < p.r && j0 + cidx < p.n) ? bf16f(p.A[(size_t)k * p.n + j0 + cidx]) : 0.0f;
                }
                __syncthreads();
#pragma unroll
                for (int t = 0; t < kTok; ++t) {
                    const float4 b4 = *reinterpret_cast<const float4 *>(&gs[t][ty * 4]);
                    const float4 a4 = *reinterpret_cast<const float4 *>(&xs[t][tx * 4]);
                    const float bv[4] = {b4.x, b4.y, b4.z, b4.w}, av[4] = {a4.x, a4.y, a4.z, a4.w};
#pragma unroll
                    for (int a = 0; a < 4; ++a)
#pragma unroll
                        for (int b = 0; b < 4; ++b) sc[a][b] = fmaf(bv[a], av[b], sc[a][b]);
                }
                __syncthreads();
            }
        }
        // ---- dS = (g^T x) (.) L[Q]   (QAT: (.) (L[Q] - W (/) S))
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int i = i0 + ty * 4 + a, j = j0 + tx * 4 + b;
                float lv = 0.0f;
                if (i < p.m && j < p.n) {
                    lv = lv_s[read_code(p.q, row_bytes, i, j, p.bits)];
                    if (p.W) {
                        lv = sc[a][b] != 0.0f ? lv - bf16f(p.W[(size_t)i * p.n + j]) / sc[a][b] : 0.0f;
                        if (write_dW) p.dW[(size_t)i * p.n + j] = c[a][b];
                    }
                }
                ds[ty * 4 + a][tx * 4 + b] = c[a][b] * lv;
            }
        // ---- the factor slice that folds the tile: A[:, j0 ..] (ROLE 0) or B[i0 .., :] (ROLE 1), zero padded
        for (int e = tid; e < r4 * kT; e += kBwThreads) {
            const int k = e / kT, cidx = e % kT;
            uint16_t v = 0;
            if (k < p.r) {
                if (ROLE == 0) { if (j0 + cidx < p.n) v = p.A[(size_t)k * p.n + j0 + cidx]; }
                else { if (i0 + cidx < p.m) v = p.B[(size_t)(i0 + cidx) * p.r + k]; }
            }
            fs[k][cidx] = v;
        }
        __syncthreads();
        // ---- fold: ROLE 0: dB[i][k] += sum_j dS[i][j] A[k][j];  ROLE 1: dA[k][j] += sum_i B[i][k] dS[i][j]
#pragma unroll
        for (int a = 0; a < kAccMax; ++a) {
            if (a >= nacc4) break;
            const int e = tid + kBwThreads * a;
            float s = acc[a];
            if (ROLE == 0) {
                const int i = e / r4, k = e % r4;
#pragma unroll 8
                for (int j = 0; j < kT; ++j) s = fmaf(ds[i][j], bf16f(fs[k][j]), s);
            } else {
                const int k = e / kT, j = e % kT;
#pragma unroll 8
                for (int i = 0; i < kT; ++i) s = fmaf(bf16f(fs[k][i]), ds[i][j], s);
            }
            acc[a] = s;
        }
        __syncthreads();
    }
#pragma unroll
    for (int a = 0; a < kAccMax; ++a) {
        if (a >= nacc4) break;
        const int e = tid + kBwThreads * a;
        if (ROLE == 0) {
            const int i = own0 + e / r4, k = e % r4;
            if (p.dB && i < p.m && k < p.r) p.dB[(size_t)i * p.r + k] = acc[a];
        } else {
            const int k = e / kT, j = own0 + e % kT;
            if (p.dA && k < p.r && j < p.n) p.dA[(size_t)k * p.n + j] = acc[a];
        }
    }
}

// Schedule "tiles": CTA (jt, it) handles rows it * 64 .. and columns jt * 64 .. of W.
//   part_dB[jt][i][k4]  (k4 < r4: r rounded up to a multiple of 4) and part_dA[it][k4][j]
__global__ void __launch_bounds__(kBwThreads) lords_backward_tile_kernel(const BwParams p, float *__restrict__ part_dB,
                                                                         float *__restrict__ part_dA)
{
    __shared__ __align__(16) float gs[kTok][kT];
    __shared__ __align__(16) float xs[kTok][kT];
    __shared__ float ds[kT][kT + 1];
    __shared__ uint16_t fs[kRMaxBw][kT + 2];
    __shared__ float lv_s[16];

    const int tid = threadIdx.x;
    if (tid < 16) lv_s[tid] = p.levels[tid];       // read after the first __syncthreads below
    const int ty = tid >> 4, tx = tid & 15;
    const int jt = blockIdx.x, it = blockIdx.y;
    const int i0 = it * kT, j0 = jt * kT;
    const size_t row_bytes = (size_t)p.n * p.bits / 8;
    const int r4 = (p.r + 3) & ~3;
    const int nacc4 = r4 * kT / kBwThreads;

    float c[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) c[a][b] = 0.0f;
    for (int t0 = 0; t0 < p.M; t0 += kTok) {
        for (int e = tid; e < kTok * kT; e += kBwThreads) {
            const int t = t0 + e / kT, cidx = e % kT;
            gs[e / kT][cidx] = (t < p.M && i0 + cidx < p.m) ? bf16f(p.g[(size_t)t * p.m + i0 + cidx]) : 0.0f;
            xs[e / kT][cidx] = (t < p.M && j0 + cidx < p.n) ? bf16f(p.x[(size_t)t * p.n + j0 + cidx]) : 0.0f;
        }
        __syncthreads();
#pragma unroll
        for (int t = 0; t < kTok; ++t) {
            const float4 g4 = *reinterpret_cast<const float4 *>(&gs[t][ty * 4]);
            const float4 x4 = *reinterpret_cast<const float4 *>(&xs[t][tx * 4]);
            const float gv[4] = {g4.x, g4.y, g4.z, g4.w}, xv[4] = {x4.x, x4.y, x4.z, x4.w};
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) c[a][b] = fmaf(gv[a], xv[b], c[a][b]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int i = i0 + ty * 4 + a, j = j0 + tx * 4 + b;
            float lv = 0.0f;
            if (i < p.m && j < p.n) lv = lv_s[read_code(p.q, row_bytes, i, j, p.bits)];
            ds[ty * 4 + a][tx * 4 + b] = c[a][b] * lv;
        }
    if (part_dB) {
        for (int e = tid; e < r4 * kT; e += kBwThreads) {           // A[k][j0 ..], zero padded
            const int k = e / kT, cidx = e % kT;
            fs[k][cidx] = (k < p.r && j0 + cidx < p.n) ? p.A[(size_t)k * p.n + j0 + cidx] : (uint16_t)0;
        }
        __syncthreads();
        float *out = part_dB + ((size_t)jt * p.m + i0) * r4;
        for (int a = 0; a < nacc4; ++a) {
            const int e = tid + kBwThreads * a, i = e / r4, k = e % r4;
            float s = 0.0f;
#pragma unroll 8
            for (int j = 0; j < kT; ++j) s = fmaf(ds[i][j], bf16f(fs[k][j]), s);
            if (i0 + i < p.m) out[(size_t)i * r4 + k] = s;
        }
    }
    __syncthreads();
    if (part_dA) {
        for (int e = tid; e < r4 * kT; e += kBwThreads) {           // B[i0 ..][k] stored [k][i], zero padded
            const int k = e / kT, cidx = e % kT;
            fs[k][cidx] = (k < p.r && i0 + cidx < p.m) ? p.B[(size_t)(i0 + cidx) * p.r + k] : (uint16_t)0;
        }
        __syncthreads();
        float *out = part_dA + (size_t)it * r4 * p.n + j0;
        for (int a = 0; a < nacc4; ++a) {
            const int e = tid + kBwThreads * a, k = e / kT, j = e % kT;
            float s = 0.0f;
#pragma unroll 8
            for (int i = 0; i < kT; ++i) s = fmaf(bf16f(fs[k][i]), ds[i][j], s);
            if (j0 + j < p.n) out[(size_t)k * p.n + j] = s;
        }
    }
}

// Schedule "tensor": CTA (jt, it) handles rows it * 128 .. and columns jt * 64 .. of W.
//   G[128 x 64] = sum_t g[t][i] x[t][j]:  both operands are MN-major in shared memory (a row of the tile
//   is one token: 64 consecutive rows or columns of W), K = 16 tokens per MMA, 64 tokens per stage.
// Warps 0..7: epilogue (level multiply, folds); 8: TMEM allocation and MMA issue; 9: TMA producer.
constexpr int kTcRows = 128, kTcCols = 64, kTcTok = 64, kTcStages = 3;
constexpr int kTcThreads = 320;
constexpr int kTcGAtom = kTcTok * 128;                        // 64 tokens x 64 rows of W, bf16
constexpr int kTcStage = 2 * kTcGAtom + kTcTok * 128;         // g: two atoms, x: one
constexpr uint32_t kTcTmemCols = 64;
// epilogue buffers (floats): rows of the dS tile and of the A slice are 68 floats apart, rows of the B slice
// (stored [rank][row]) 132: multiples of four, so that four neighbouring values are one 16-byte word, and with
// 16-byte words of consecutive rows in different banks
constexpr int kTcDsPitch = kTcCols + 4, kTcFbPitch = kTcRows + 4;

struct alignas(64) BwTcParams {
    CUtensorMap tm_g;     // bf16 [M][m], box {64, 64}, 128-byte swizzle (tokens past M read as zero)
    CUtensorMap tm_x;     // bf16 [M][n], box {64, 64}, 128-byte swizzle
    BwParams b;
    float *part_dB;       // [n / 64 tiles][m][r4]
    float *part_dA;       // [m / 128 tiles][r4][n]
    int *status;
    // quantisation-aware training (Eq. 4-5): the latent weight and, optionally, where dL/dW goes
    const uint16_t *W;    // bf16 [m][n]
    float *dW;            // float [m][n] or null
    // QAT with a rank that is a multiple of 8 up to 64: S = B_tile A_tile by a scale MMA (Eq. 3), as in the forward kernels
    CUtensorMap tm_b;     // bf16 [m][r], box {64 ranks, 128 rows}, 128-byte swizzle (ranks past r read as zero)
    CUtensorMap tm_a;     // bf16 [r][n], box {64 columns, ceil16(r) ranks}, 128-byte swizzle
    int scale_mma;
};

constexpr int kTcBTile = kTcRows * 128;                       // scale MMA: B[128 rows][64 ranks] bf16
constexpr int kTcATile = 64 * 128;                            // scale MMA: A[64 ranks][64 columns] bf16

__host__ __device__ constexpr int bw_tc_smem(int r4, bool qat)
{
    // the epilogue's buffers (dS tile, the two factor slices) reuse the stages once the MMAs are done;
    // the operand tiles of the scale MMA (QAT) lie behind the barriers, on a 1024-byte boundary of their own
    const int stages = kTcStages * kTcStage;
    const int epi = kTcRows * kTcDsPitch * 4 + r4 * kTcDsPitch * 4 + r4 * kTcFbPitch * 4;
    return 1024 + (stages > epi ? stages : epi) + 256 + (qat ? 1024 + kTcBTile + kTcATile : 0);
}

// QAT: the tile of g^T x is dL/dW^ itself (Eq. 4: stored as dL/dW if asked for), and the factor of
// dL/dS is Q - W (/) S instead of Q (Eq. 5), with S = B A rebuilt per element from the factor slices.
template <bool QAT>
__global__ void __launch_bounds__(kTcThreads, 2) lords_backward_tc_kernel(const __grid_constant__ BwTcParams p)
{
    extern __shared__ uint8_t tc_smem_raw[];
    const uint32_t base = (smem_u32(tc_smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = tc_smem_raw + (base - smem_u32(tc_smem_raw));
    const int r4 = (p.b.r + 3) & ~3;
    const int stages_bytes = kTcStages * kTcStage;
    const int epi_bytes = kTcRows * kTcDsPitch * 4 + r4 * kTcDsPitch * 4 + r4 * kTcFbPitch * 4;
    const uint32_t bars = base + (uint32_t)(stages_bytes > epi_bytes ? stages_bytes : epi_bytes);
    const uint32_t bar_full = bars, bar_empty = bars + 8 * kTcStages, bar_acc = bar_empty + 8 * kTcStages;
    const uint32_t tmem_slot = bar_acc + 8;
    const uint32_t bar_s_full = bar_acc + 16, bar_s_done = bar_acc + 24;     // scale MMA (QAT): operand tiles landed, S complete
    const uint32_t s_btile = (bars + 256u + 1023u) & ~1023u, s_atile = s_btile + kTcBTile;
    const bool scale_mma = QAT && p.scale_mma != 0;
    constexpr uint32_t kTmemCols = QAT ? 2 * kTcTmemCols : kTcTmemCols;     // QAT: S in the columns behind the accumulator
    const int r16 = (p.b.r + 15) & ~15;
    // the level table in shared memory (16 floats behind the barriers): a lookup by a per-thread code is one
    // conflict-free read there, where the same lookup in the kernel parameters is replayed once per distinct code
    float *levels_s = reinterpret_cast<float *>(base_ptr + (bars - base) + 128);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int jt = blockIdx.x, it = blockIdx.y;
    const int i0 = it * kTcRows, j0 = jt * kTcCols;
    const int chunks = (p.b.M + kTcTok - 1) / kTcTok;
    const int *status = p.status;
    bool failed = false;

    if (tid == 0) {
        for (int s = 0; s < kTcStages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        mbar_init(bar_acc, 1);
        mbar_init(bar_s_full, 1);
        mbar_init(bar_s_done, 1);
        fence_mbar_init();
    }
    if (tid >= 32 && tid < 48) levels_s[tid - 32] = p.b.levels[tid - 32];
    if (warp == 8) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

    if (warp == 9) {
        if (lane == 0) {
            tma_prefetch_desc(&p.tm_g);
            tma_prefetch_desc(&p.tm_x);
            if (scale_mma) {
                mbar_expect_tx(bar_s_full, (uint32_t)(kTcBTile + r16 * 128));
                tma_load_2d(s_btile, &p.tm_b, 0, i0, bar_s_full);
                tma_load_2d(s_atile, &p.tm_a, j0, 0, bar_s_full);
            }
            for (int c = 0; c < chunks; ++c) {
                const int s = c % kTcStages;
                if (c >= kTcStages && !mbar_wait(bar_empty + 8 * s, (uint32_t)((c / kTcStages - 1) & 1), status, 41)) { failed = true; break; }
                const uint32_t bar = bar_full + 8 * s, st0 = base + (uint32_t)(s * kTcStage);
                mbar_expect_tx(bar, (uint32_t)kTcStage);
                tma_load_2d(st0, &p.tm_g, i0, c * kTcTok, bar);
                tma_load_2d(st0 + kTcGAtom, &p.tm_g, i0 + 64, c * kTcTok, bar);
                tma_load_2d(st0 + 2 * kTcGAtom, &p.tm_x, j0, c * kTcTok, bar);
            }
        }
    } else if (warp == 8) {
        constexpr uint32_t idesc = umma_idesc_f16(1, 1, 1, kTcRows, kTcCols);     // bf16, both operands MN-major
        const uint32_t a_hi = (uint32_t)(umma_desc_sw128(0, 1024, (uint32_t)kTcGAtom) >> 32);
        const uint32_t a_lo0 = (uint32_t)umma_desc_sw128(0, 1024, (uint32_t)kTcGAtom) | ((base & 0x3FFFFu) >> 4);
        const uint32_t b_hi = (uint32_t)(umma_desc_sw128(0, 1024, 16) >> 32);
        const uint32_t b_lo0 = (uint32_t)umma_desc_sw128(0, 1024, 16) | (((base + 2 * kTcGAtom) & 0x3FFFFu) >> 4);
        if (scale_mma) {
            // S[128 x 64] = B_tile (K-major: a row is one row of B, 16 ranks = 32 bytes) * A_tile (MN-major: a row is one
            // rank, 16 ranks = 16 rows of 128 bytes), one MMA per 16 ranks, into the columns behind the accumulator
            constexpr uint32_t idesc_s = umma_idesc_f16(1, 0, 1, kTcRows, kTcCols);
            if (!mbar_wait(bar_s_full, 0, status, 44)) failed = true;
            tc_fence_after_sync();
            if (lane == 0 && !failed) {
                const uint32_t sb_lo = (uint32_t)umma_desc_sw128(0, 1024, 16) | ((s_btile & 0x3FFFFu) >> 4);
                const uint32_t sa_lo = (uint32_t)umma_desc_sw128(0, 1024, 16) | ((s_atile & 0x3FFFFu) >> 4);
                for (int k = 0; k < r16 / 16; ++k)
                    umma_f16_ss(tmem_base + kTcTmemCols, umma_desc_pack(sb_lo + k * 2, b_hi), umma_desc_pack(sa_lo + k * 128, b_hi),
                                idesc_s, k > 0 ? 1u : 0u);
                umma_commit(bar_s_done);
            }
            __syncwarp();
        }
        for (int c = 0; c < chunks && !failed; ++c) {
            const int s = c % kTcStages;
            if (!mbar_wait(bar_full + 8 * s, (uint32_t)((c / kTcStages) & 1), status, 42)) { failed = true; break; }
            tc_fence_after_sync();
            if (lane == 0) {
                const uint32_t off = (uint32_t)((s * kTcStage) >> 4);
#pragma unroll
                for (int k = 0; k < kTcTok / 16; ++k)      // 16 tokens = 16 rows of 128 bytes
                    umma_f16_ss(tmem_base, umma_desc_pack(a_lo0 + off + k * 128, a_hi), umma_desc_pack(b_lo0 + off + k * 128, b_hi),
                                idesc, (c > 0 || k > 0) ? 1u : 0u);
                umma_commit(bar_empty + 8 * s);
                if (c == chunks - 1) umma_commit(bar_acc);
            }
            __syncwarp();
        }
    } else {
        // ---- epilogue: thread = (row quadrant q, column half ch): row i0 + q * 32 + lane, 32 columns
        const int q = warp & 3, ch = warp >> 2;
        const int ri = q * 32 + lane, i = i0 + ri;
        // the dS tile and the factor slices (widened to fp32)
        float (*ds)[kTcDsPitch] = reinterpret_cast<float (*)[kTcDsPitch]>(base_ptr);
        float (*fa)[kTcDsPitch] = reinterpret_cast<float (*)[kTcDsPitch]>(base_ptr + kTcRows * kTcDsPitch * 4);
        float (*fb)[kTcFbPitch] =
            reinterpret_cast<float (*)[kTcFbPitch]>(base_ptr + kTcRows * kTcDsPitch * 4 + r4 * kTcDsPitch * 4);
        // What the epilogue needs from global memory does not depend on the tile product: the thread's codes and, for
        // ranks that are multiples of 8 up to 32 (one 16-byte piece of the A slice and two of the B slice per thread),
        // the factor slices are requested before the wait for the accumulator and parked in registers.
        const int et = tid;                                       // 0 .. 255
        const size_t row_bytes = (size_t)p.b.n * p.b.bits / 8;
        const int jc = j0 + ch * 32, bits = p.b.bits;
        // the thread's 32 codes are `bits` consecutive 32-bit words of its row when the group lies
        // inside the row and the row pitch keeps it word-aligned; otherwise code by code
        const bool whole_shape = i < p.b.m && jc + 32 <= p.b.n && (row_bytes & 3) == 0;
        uint32_t cw[5] = {0u, 0u, 0u, 0u, 0u};
        if (whole_shape) {
            const uint32_t *src = reinterpret_cast<const uint32_t *>(p.b.q + (size_t)i * row_bytes + (size_t)jc * bits / 8);
#pragma unroll
            for (int w = 0; w < 4; ++w)
                if (w < bits) cw[w] = __ldg(src + w);
        }
        const bool parked = (p.b.r & 7) == 0 && r4 <= 32;
        uint4 park_a = make_uint4(0u, 0u, 0u, 0u), park_b[2] = {park_a, park_a};
        if (parked) {
            const int k = et / (kTcCols / 8), c8 = 8 * (et % (kTcCols / 8));
            if (k < p.b.r && j0 + c8 < p.b.n) park_a = __ldg(reinterpret_cast<const uint4 *>(p.b.A + (size_t)k * p.b.n + j0 + c8));
            const int per_row = p.b.r / 8;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int e = et + 256 * h, cidx = e / per_row, k8 = 8 * (e % per_row);
                if (e < kTcRows * per_row && i0 + cidx < p.b.m)
                    park_b[h] = __ldg(reinterpret_cast<const uint4 *>(p.b.B + (size_t)(i0 + cidx) * p.b.r + k8));
            }
        }
        // QAT: the thread's 32 latent weights (64 bytes of its row; n is a multiple of 8, so a group of eight is whole)
        uint4 wq[QAT ? 4 : 1];
        if constexpr (QAT) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                wq[v] = make_uint4(0u, 0u, 0u, 0u);
                if (i < p.b.m && jc + 8 * v < p.b.n) wq[v] = __ldg(reinterpret_cast<const uint4 *>(p.W + (size_t)i * p.b.n + jc + 8 * v));
            }
        }
        const bool ok = __all_sync(0xffffffffu, mbar_wait(bar_acc, 0, status, 43));
        if (!ok) failed = true;
        tc_fence_after_sync();
        uint32_t gacc[32];
        if (ok) {
            tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(ch * 32), gacc);
            tmem_wait_ld();
        }
        // every MMA has completed (the accumulator barrier), so every stage has been read: the stages'
        // memory now holds the factor slices and the dS tile
        auto store_a8 = [&](int k, int c8, const uint4 &v) {
            *reinterpret_cast<float4 *>(&fa[k][c8]) = make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u),
                                                                  __uint_as_float(v.y << 16), __uint_as_float(v.y & 0xFFFF0000u));
            *reinterpret_cast<float4 *>(&fa[k][c8 + 4]) = make_float4(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xFFFF0000u),
                                                                      __uint_as_float(v.w << 16), __uint_as_float(v.w & 0xFFFF0000u));
        };
        auto store_b8 = [&](int cidx, int k8, const uint4 &v) {
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                fb[k8 + 2 * h][cidx] = __uint_as_float(w[h] << 16);
                fb[k8 + 2 * h + 1][cidx] = __uint_as_float(w[h] & 0xFFFF0000u);
            }
        };
        auto load_slices = [&]() {
            if (parked) {
                if (et < r4 * (kTcCols / 8)) store_a8(et / (kTcCols / 8), 8 * (et % (kTcCols / 8)), park_a);
                const int per_row = p.b.r / 8;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int e = et + 256 * h;
                    if (e < kTcRows * per_row) store_b8(e / per_row, 8 * (e % per_row), park_b[h]);
                }
                return;
            }
            // A[k][j0 ..]: eight columns (16 bytes) per load -- n is a multiple of 8 on this schedule, so a group
            // of eight columns is whole and aligned
            for (int e = et; e < r4 * (kTcCols / 8); e += 256) {
                const int k = e / (kTcCols / 8), c8 = 8 * (e % (kTcCols / 8));
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (k < p.b.r && j0 + c8 < p.b.n) v = __ldg(reinterpret_cast<const uint4 *>(p.b.A + (size_t)k * p.b.n + j0 + c8));
                store_a8(k, c8, v);
            }
            // B[i0 ..][k] stored [k][i]
            if ((p.b.r & 7) == 0) {                                   // rows of B are 16-byte multiples: eight ranks per load
                const int per_row = p.b.r / 8;
                for (int e = et; e < kTcRows * per_row; e += 256) {
                    const int cidx = e / per_row, k8 = 8 * (e % per_row);
                    uint4 v = make_uint4(0u, 0u, 0u, 0u);
                    if (i0 + cidx < p.b.m) v = __ldg(reinterpret_cast<const uint4 *>(p.b.B + (size_t)(i0 + cidx) * p.b.r + k8));
                    store_b8(cidx, k8, v);
                }
            } else {
                for (int e = et; e < r4 * kTcRows; e += 256) {        // neighbouring threads read one row of B
                    const int cidx = e / r4, k = e % r4;
                    fb[k][cidx] = (k < p.b.r && i0 + cidx < p.b.m) ? bf16f(p.b.B[(size_t)(i0 + cidx) * p.b.r + k]) : 0.0f;
                }
            }
        };
        if constexpr (QAT) load_slices();                         // S is rebuilt from them below
        const bool whole = ok && whole_shape;
        // QAT: W / S per element (0 where S is 0, and the level is dropped there too: no gradient)
        float quot[QAT ? 32 : 1];
        bool live[QAT ? 32 : 1];
        if constexpr (QAT) {
            if (p.dW && ok && i < p.b.m) {                        // Eq. 4: dL/dW = dL/dW^
#pragma unroll
                for (int c4 = 0; c4 < 32; c4 += 4)
                    if (jc + c4 < p.b.n)
                        *reinterpret_cast<float4 *>(p.dW + (size_t)i * p.b.n + jc + c4) =
                            make_float4(__uint_as_float(gacc[c4]), __uint_as_float(gacc[c4 + 1]), __uint_as_float(gacc[c4 + 2]),
                                        __uint_as_float(gacc[c4 + 3]));
            }
            float sv[32];
            if (scale_mma) {
                // S of the thread's row and columns from the scale MMA (complete long before the tile product)
                if (!__all_sync(0xffffffffu, mbar_wait(bar_s_done, 0, status, 45))) failed = true;
                tc_fence_after_sync();
                uint32_t sraw[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + kTcTmemCols + (uint32_t)(ch * 32), sraw);
                tmem_wait_ld();
#pragma unroll
                for (int cidx = 0; cidx < 32; ++cidx) sv[cidx] = failed ? 0.0f : __uint_as_float(sraw[cidx]);
            } else {
                asm volatile("bar.sync 1, 256;" ::: "memory");    // the factor slices are in place
#pragma unroll
                for (int cidx = 0; cidx < 32; ++cidx) sv[cidx] = 0.0f;
                for (int k = 0; k < p.b.r; ++k) {
                    const float bk = fb[k][ri];
#pragma unroll
                    for (int cidx = 0; cidx < 32; ++cidx) sv[cidx] = fmaf(bk, fa[k][ch * 32 + cidx], sv[cidx]);
                }
            }
#pragma unroll
            for (int cidx = 0; cidx < 32; ++cidx) {
                const uint4 &wv = wq[cidx / 8];
                const uint32_t ww = (cidx % 8) / 2 == 0 ? wv.x : (cidx % 8) / 2 == 1 ? wv.y : (cidx % 8) / 2 == 2 ? wv.z : wv.w;
                const float w = __uint_as_float((cidx & 1) ? (ww & 0xFFFF0000u) : (ww << 16));
                live[cidx] = sv[cidx] != 0.0f;
                // w / S by a reciprocal and one residual correction: exact whenever the quotient is representable
                // (a weight that its code reproduces exactly gets the factor 0), a rounding error otherwise
                const float rc = __fdividef(1.0f, sv[cidx]);
                float qv = w * rc;
                qv = fmaf(fmaf(-qv, sv[cidx], w), rc, qv);
                quot[cidx] = live[cidx] ? qv : 0.0f;
            }
        }
        auto factor = [&](int cidx, float level) -> float {
            if constexpr (QAT) return live[cidx] ? level - quot[cidx] : 0.0f;
            else return level;
        };
        if (whole) {
            // the positions of the codes inside the words are compile-time constants for each width
            auto levels_of = [&](auto width) {
                constexpr int W = decltype(width)::value;
                float dv[4];
#pragma unroll
                for (int cidx = 0; cidx < 32; ++cidx) {
                    constexpr uint32_t mask = (1u << W) - 1u;
                    const int bit = cidx * W, w = bit >> 5, sh = bit & 31;
                    uint32_t code = cw[w] >> sh;
                    if (sh + W > 32) code |= cw[w + 1] << (32 - sh);
                    dv[cidx & 3] = __uint_as_float(gacc[cidx]) * factor(cidx, levels_s[code & mask]);
                    if ((cidx & 3) == 3)
                        *reinterpret_cast<float4 *>(&ds[ri][ch * 32 + cidx - 3]) = make_float4(dv[0], dv[1], dv[2], dv[3]);
                }
            };
            if (bits == 4) levels_of(std::integral_constant<int, 4>{});
            else if (bits == 3) levels_of(std::integral_constant<int, 3>{});
            else levels_of(std::integral_constant<int, 2>{});
        } else {
#pragma unroll
            for (int cidx = 0; cidx < 32; ++cidx) {
                const int j = jc + cidx;
                float v = 0.0f;
                if (ok && i < p.b.m && j < p.b.n)
                    v = __uint_as_float(gacc[cidx]) * factor(cidx, levels_s[read_code(p.b.q, row_bytes, i, j, bits)]);
                ds[ri][ch * 32 + cidx] = v;
            }
        }
        if constexpr (!QAT) load_slices();
        asm volatile("bar.sync 1, 256;" ::: "memory");
        // The folds, register-blocked so that a 16-byte word read from shared memory feeds 16 (dB) or 8 (dA)
        // multiply-adds.  Each output is one thread's sum in index order.
        if (p.part_dB) {
            // dB[i][k] = sum_j dS[i][j] A[k][j]: lane = rows lane + 32 a, warp = ranks 4 kg .. 4 kg + 3 (kg = warp, warp + 8, ..)
            float *out = p.part_dB + ((size_t)jt * p.b.m + i0) * r4;
            for (int kg = warp; kg < r4 / 4; kg += 8) {
                const int k0 = 4 * kg;
                float acc[4][4];
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int b = 0; b < 4; ++b) acc[a][b] = 0.0f;
#pragma unroll 2
                for (int j4 = 0; j4 < kTcCols / 4; ++j4) {
                    float4 d[4], w[4];
#pragma unroll
                    for (int a = 0; a < 4; ++a) d[a] = *reinterpret_cast<const float4 *>(&ds[lane + 32 * a][4 * j4]);
#pragma unroll
                    for (int b = 0; b < 4; ++b) w[b] = *reinterpret_cast<const float4 *>(&fa[k0 + b][4 * j4]);
#pragma unroll
                    for (int a = 0; a < 4; ++a)
#pragma unroll
                        for (int b = 0; b < 4; ++b) {
                            acc[a][b] = fmaf(d[a].x, w[b].x, acc[a][b]);
                            acc[a][b] = fmaf(d[a].y, w[b].y, acc[a][b]);
                            acc[a][b] = fmaf(d[a].z, w[b].z, acc[a][b]);
                            acc[a][b] = fmaf(d[a].w, w[b].w, acc[a][b]);
                        }
                }
#pragma unroll
                for (int a = 0; a < 4; ++a) {
                    const int ii = lane + 32 * a;
                    if (i0 + ii < p.b.m)
                        *reinterpret_cast<float4 *>(&out[(size_t)ii * r4 + k0]) = make_float4(acc[a][0], acc[a][1], acc[a][2], acc[a][3]);
                }
            }
        }
        if (p.part_dA) {
            // dA[k][j] = sum_i B[i][k] dS[i][j]: a thread takes 4 ranks x 4 columns over one half of the tile's rows
            // (warps 0..3: rows 0..63, warps 4..7: rows 64..127); the upper half parks its sums in shared memory
            // (the A slice's, which the dB fold is done with after the barrier), the lower half adds them to its own.
            asm volatile("bar.sync 1, 256;" ::: "memory");
            float *out = p.part_dA + (size_t)it * r4 * p.b.n + j0;
            float *park = &fa[0][0];                                  // [r4][64] floats
            const int half = warp >> 2, jq = 4 * (lane & 15), ibase = 64 * half;
            const int blocks = r4 / 4;
            for (int kb0 = 0; kb0 < blocks; kb0 += 8) {               // the same trip count for every thread
                const int kb = kb0 + 2 * (warp & 3) + (lane >> 4);
                const bool active = kb < blocks;
                const int k0 = 4 * (active ? kb : 0);
                float acc[4][4];
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[b][0] = acc[b][1] = acc[b][2] = acc[b][3] = 0.0f;
                if (active) {
#pragma unroll 4
                    for (int i2 = 0; i2 < 32; ++i2) {
                        const int ii = ibase + 2 * i2;
                        const float4 d0 = *reinterpret_cast<const float4 *>(&ds[ii][jq]);
                        const float4 d1 = *reinterpret_cast<const float4 *>(&ds[ii + 1][jq]);
#pragma unroll
                        for (int b = 0; b < 4; ++b) {
                            const float2 bv = *reinterpret_cast<const float2 *>(&fb[k0 + b][ii]);
                            acc[b][0] = fmaf(bv.x, d0.x, acc[b][0]);
                            acc[b][1] = fmaf(bv.x, d0.y, acc[b][1]);
                            acc[b][2] = fmaf(bv.x, d0.z, acc[b][2]);
                            acc[b][3] = fmaf(bv.x, d0.w, acc[b][3]);
                            acc[b][0] = fmaf(bv.y, d1.x, acc[b][0]);
                            acc[b][1] = fmaf(bv.y, d1.y, acc[b][1]);
                            acc[b][2] = fmaf(bv.y, d1.z, acc[b][2]);
                            acc[b][3] = fmaf(bv.y, d1.w, acc[b][3]);
                        }
                    }
                    if (half == 1) {
#pragma unroll
                        for (int b = 0; b < 4; ++b)
                            *reinterpret_cast<float4 *>(&park[(k0 + b) * kTcCols + jq]) = make_float4(acc[b][0], acc[b][1], acc[b][2], acc[b][3]);
                    }
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (active && half == 0 && j0 + jq < p.b.n) {        // n is a multiple of 8 on this schedule: a group of four columns is whole
#pragma unroll
                    for (int b = 0; b < 4; ++b) {
                        const float4 u = *reinterpret_cast<const float4 *>(&park[(k0 + b) * kTcCols + jq]);
                        *reinterpret_cast<float4 *>(&out[(size_t)(k0 + b) * p.b.n + jq]) =
                            make_float4(acc[b][0] + u.x, acc[b][1] + u.y, acc[b][2] + u.z, acc[b][3] + u.w);
                    }
                }
            }
        }
    }

    if (failed) atomicExch(p.status, LORDS_ERR_TIMEOUT);
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 8) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// out[e] = sum over tiles t (in order) of part[t * stride + pos(e)], for dB (rows = m, inner = r, inner4 = r4:
// blocks below blocks_b) and for dA (rows = r, inner = inner4 = n: the other blocks) in one launch.
struct ReduceJob {
    const float *part;
    float *out;
    int tiles, rows, inner, inner4;
    size_t stride;
};

__global__ void lords_backward_reduce_kernel(const ReduceJob jb, const ReduceJob ja, int blocks_b)
{
    const bool isb = (int)blockIdx.x < blocks_b;
    const ReduceJob &j = isb ? jb : ja;
    const size_t e = (size_t)(isb ? blockIdx.x : blockIdx.x - blocks_b) * blockDim.x + threadIdx.x;
    if (e >= (size_t)j.rows * j.inner) return;
    const size_t row = e / j.inner, col = e % j.inner;
    float s = 0.0f;
    for (int t = 0; t < j.tiles; ++t) s += j.part[(size_t)t * j.stride + row * j.inner4 + col];
    j.out[e] = s;
}

// The sums of the tiles' contributions to dB ([tiles_b][m][r4]) and dA ([tiles_a][r4][n]); either may be absent.
int launch_reduce(const float *part_b, float *dB, int tiles_b, const float *part_a, float *dA, int tiles_a, int m, int n, int r, int r4,
                  cudaStream_t stream)
{
    ReduceJob jb = {part_b, dB, tiles_b, dB ? m : 0, r, r4, (size_t)m * r4};
    ReduceJob ja = {part_a, dA, tiles_a, dA ? r : 0, n, n, (size_t)r4 * n};
    const size_t nb = ((size_t)jb.rows * r + 255) / 256, na = ((size_t)ja.rows * n + 255) / 256;
    if (nb + na == 0) return LORDS_OK;
    if (nb + na > 2147483647u) return LORDS_ERR_SHAPE;
    lords_backward_reduce_kernel<<<(unsigned)(nb + na), 256, 0, stream>>>(jb, ja, (int)nb);
    LORDS_CUDA_TRY(cudaGetLastError());
    return LORDS_OK;
}

}  // namespace

int launch_transpose_codes(const uint8_t *Q, int m, int n, int bits, uint8_t *Qt, cudaStream_t stream)
{
    const dim3 grid((unsigned)((n + 127) / 128), (unsigned)((m + 31) / 32));
    if (grid.y > 65535u) return LORDS_ERR_SHAPE;
    lords_transpose_codes_kernel<<<grid, 128, 0, stream>>>(Q, Qt, m, n, bits);
    LORDS_CUDA_TRY(cudaGetLastError());
    return LORDS_OK;
}

int launch_transpose_bf16_pair(const uint16_t *src0, int rows0, int cols0, uint16_t *dst0, const uint16_t *src1, int rows1, int cols1,
                               uint16_t *dst1, cudaStream_t stream)
{
    const long long t0 = (long long)((cols0 + 31) / 32) * ((rows0 + 31) / 32), t1 = (long long)((cols1 + 31) / 32) * ((rows1 + 31) / 32);
    if (t0 + t1 > 2147483647LL) return LORDS_ERR_SHAPE;
    lords_transpose_bf16_pair_kernel<<<(unsigned)(t0 + t1), dim3(32, 8), 0, stream>>>(src0, dst0, rows0, cols0, src1, dst1, rows1, cols1, (int)t0);
    LORDS_CUDA_TRY(cudaGetLastError());
    return LORDS_OK;
}

// The tensor schedule.  W != null: the gradients of quantisation-aware training (dW may be null).
// LORDS_ERR_UNSUPPORTED when the shapes do not suit it or the workspace cannot hold the contributions.
static int launch_backward_tc(const BwParams &p, const uint16_t *W, float *dW, State &st, cudaStream_t stream)
{
    const int m = p.m, n = p.n, r = p.r, M = p.M;
    const int r4 = (r + 3) & ~3;
    const int it_t = (m + kTcRows - 1) / kTcRows, jt_t = (n + kTcCols - 1) / kTcCols;
    const size_t nb = p.dB ? (size_t)jt_t * m * r4 * sizeof(float) : 0, na = p.dA ? (size_t)it_t * r4 * n * sizeof(float) : 0;
    if (m % 8 != 0 || n % 8 != 0 || it_t > 65535 || nb + na + 256 > st.workspace_bytes) return LORDS_ERR_UNSUPPORTED;
    BwTcParams k;
    k.b = p;
    k.part_dB = p.dB ? reinterpret_cast<float *>(st.workspace) : nullptr;
    k.part_dA = p.dA ? reinterpret_cast<float *>(st.workspace + ((nb + 255) & ~(size_t)255)) : nullptr;
    k.status = st.status_word;
    k.W = W; k.dW = dW;
    if (!make_map_2d(&k.tm_g, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p.g, (uint64_t)m, (uint64_t)M, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_2d(&k.tm_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p.x, (uint64_t)n, (uint64_t)M, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B))
        return LORDS_ERR_CUDA;
    k.scale_mma = (W && (r & 7) == 0 && r <= 64) ? 1 : 0;
    k.tm_b = k.tm_g; k.tm_a = k.tm_g;                                      // placeholders when the scale MMA is not used
    if (k.scale_mma &&
        (!make_map_2d(&k.tm_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p.B, (uint64_t)r, (uint64_t)m, 64, (uint32_t)kTcRows, CU_TENSOR_MAP_SWIZZLE_128B) ||
         !make_map_2d(&k.tm_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p.A, (uint64_t)n, (uint64_t)r, 64, (uint32_t)((r + 15) & ~15), CU_TENSOR_MAP_SWIZZLE_128B)))
        return LORDS_ERR_CUDA;
    const int smem = bw_tc_smem(r4, W != nullptr);
    static bool attr_set[kMaxDevices] = {};
    const int dev = device_slot(st);
    if (!attr_set[dev]) {
        LORDS_CUDA_TRY(cudaFuncSetAttribute(lords_backward_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bw_tc_smem(kRMaxBw, false)));
        LORDS_CUDA_TRY(cudaFuncSetAttribute(lords_backward_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bw_tc_smem(kRMaxBw, true)));
        attr_set[dev] = true;
    }
    if (W) lords_backward_tc_kernel<true><<<dim3((unsigned)jt_t, (unsigned)it_t), kTcThreads, smem, stream>>>(k);
    else lords_backward_tc_kernel<false><<<dim3((unsigned)jt_t, (unsigned)it_t), kTcThreads, smem, stream>>>(k);
    LORDS_CUDA_TRY(cudaGetLastError());
    int launches = 1;
    if (p.dB || p.dA) {
        const int rc = launch_reduce(k.part_dB, p.dB, jt_t, k.part_dA, p.dA, it_t, m, n, r, r4, stream);
        if (rc != LORDS_OK) return rc;
        ++launches;
    }
    st.last_launches = launches;
    st.last_path = W ? "backward_qat_tensor" : "backward_tensor";
    return LORDS_OK;
}

int launch_backward_factors(const uint16_t *g, const uint16_t *x, const uint8_t *q, const uint16_t *B, const uint16_t *A,
                            const float *levels, int bits, int M, int m, int n, int r, float *dB, float *dA,
                            State &st, cudaStream_t stream)
{
    if (r > kRMaxBw) return LORDS_ERR_SHAPE;
    BwParams p;
    p.g = g; p.x = x; p.q = q; p.B = B; p.A = A;
    for (int c = 0; c < 16; ++c) p.levels[c] = c < (1 << bits) ? levels[c] : 0.0f;
    p.bits = bits; p.M = M; p.m = m; p.n = n; p.r = r;
    p.dB = dB; p.dA = dA;
    p.W = nullptr; p.dW = nullptr;
    int launches = 0;
    // schedule "tiles" when the workspace holds the tiles' contributions
    const int r4 = (r + 3) & ~3, it_n = (m + kT - 1) / kT, jt_n = (n + kT - 1) / kT;
    const size_t need_b = dB ? (size_t)jt_n * m * r4 * sizeof(float) : 0, need_a = dA ? (size_t)it_n * r4 * n * sizeof(float) : 0;
    // schedule "tensor": the same with 128 x 64 tiles and the tile product on the tensor cores
    if (st.forced_path == 0) {
        const int rc = launch_backward_tc(p, nullptr, nullptr, st, stream);
        if (rc != LORDS_ERR_UNSUPPORTED) return rc;
    }
    if (it_n <= 65535 && need_b + need_a + 256 <= st.workspace_bytes && st.forced_path != 1) {
        float *part_b = dB ? reinterpret_cast<float *>(st.workspace) : nullptr;
        float *part_a = dA ? reinterpret_cast<float *>(st.workspace + ((need_b + 255) & ~(size_t)255)) : nullptr;
        lords_backward_tile_kernel<<<dim3((unsigned)jt_n, (unsigned)it_n), kBwThreads, 0, stream>>>(p, part_b, part_a);
        LORDS_CUDA_TRY(cudaGetLastError());
        ++launches;
        {
            const int rc = launch_reduce(part_b, dB, jt_n, part_a, dA, it_n, m, n, r, r4, stream);
            if (rc != LORDS_OK) return rc;
            ++launches;
        }
        st.last_launches = launches;
        st.last_path = "backward_tiles";
        return LORDS_OK;
    }
    if (dB) {
        lords_backward_factors_kernel<0><<<(unsigned)((m + kT - 1) / kT), kBwThreads, 0, stream>>>(p, 0);
        LORDS_CUDA_TRY(cudaGetLastError());
        ++launches;
    }
    if (dA) {
        lords_backward_factors_kernel<1><<<(unsigned)((n + kT - 1) / kT), kBwThreads, 0, stream>>>(p, 0);
        LORDS_CUDA_TRY(cudaGetLastError());
        ++launches;
    }
    st.last_launches = launches;
    st.last_path = "backward_walk";
    return LORDS_OK;
}

// Straight-through gradients of quantisation-aware training (Eq. 4-5): the tensor schedule where the shapes
// and the workspace allow it, else the walk (any shape, no scratch memory; g^T x is formed once per
// requested factor gradient).
int launch_backward_qat(const uint16_t *g, const uint16_t *x, const uint16_t *W, const uint8_t *q, const uint16_t *B,
                        const uint16_t *A, const float *levels, int bits, int M, int m, int n, int r, float *dW, float *dB,
                        float *dA, State &st, cudaStream_t stream)
{
    if (r > kRMaxBw) return LORDS_ERR_SHAPE;
    BwParams p;
    p.g = g; p.x = x; p.q = q; p.B = B; p.A = A;
    for (int c = 0; c < 16; ++c) p.levels[c] = c < (1 << bits) ? levels[c] : 0.0f;
    p.bits = bits; p.M = M; p.m = m; p.n = n; p.r = r;
    p.dB = dB; p.dA = dA;
    p.W = nullptr; p.dW = nullptr;                       // the tensor schedule takes them as arguments
    if (st.forced_path == 0) {
        const int rc = launch_backward_tc(p, W, dW, st, stream);
        if (rc != LORDS_ERR_UNSUPPORTED) return rc;
    }
    p.W = W; p.dW = dW;
    int launches = 0;
    const bool rows_pass = dB || !dA;                    // dL/dW alone is written by the row pass
    if (rows_pass) {
        lords_backward_factors_kernel<0><<<(unsigned)((m + kT - 1) / kT), kBwThreads, 0, stream>>>(p, dW ? 1 : 0);
        LORDS_CUDA_TRY(cudaGetLastError());
        ++launches;
    }
    if (dA) {
        lords_backward_factors_kernel<1><<<(unsigned)((n + kT - 1) / kT), kBwThreads, 0, stream>>>(p, dW && !rows_pass ? 1 : 0);
        LORDS_CUDA_TRY(cudaGetLastError());
        ++launches;
    }
    st.last_launches = launches;
    st.last_path = "backward_qat_walk";
    return LORDS_OK;
}

}  // namespace lords
