// Comparators for the paper's efficiency claims (Sec. 4.4, Table 6): what a block-scaled layer with an
// additive low-rank adapter has to run on top of its dequantise-and-multiply, written for the same
// GPU so that the ratios can be restated here.
//
//     y = x W_block^T + (x A_l^T) B_l^T        W_block = L[Q] (.) (s (x) 1)   (Eq. 2),   A_l: r x n,  B_l: m x r
//
// The block-scaled product is the 16-token decode kernel in its block-scale instantiation
// (lords_decode16.cu); the adapter cannot be merged into 4-bit weights (Sec. 3.4), so it costs two more
// launches: u = x A_l^T (M x r), then y += u B_l^T.  Both are small, memory-bound CUDA-core kernels in
// fp32 over exactly widened bf16 inputs, each output summed by one thread or one block in a fixed order.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "lords_internal.h"

namespace lords {

namespace {

__device__ __forceinline__ float bf16f(uint16_t h) { return __uint_as_float((uint32_t)h << 16); }

constexpr int kMaxTok = 16;

// u[t][k] = sum_j x[t][j] A_l[k][j]: one block per adapter rank k, all tokens at once.  A thread takes groups of
// eight columns (one 16-byte load of A_l and one of x per token), all requested before the first use; columns
// that do not fill a group of eight (or rows that are not 16-byte aligned) are taken one by one.
__global__ void __launch_bounds__(256) lords_adapter_down_kernel(const uint16_t *__restrict__ x, const uint16_t *__restrict__ Al,
                                                                 float *__restrict__ u, int M, int n, int r)
{
    __shared__ float red[8][kMaxTok];
    const int k = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float acc[kMaxTok];
#pragma unroll
    for (int t = 0; t < kMaxTok; ++t) acc[t] = 0.0f;
    const bool vec = n % 8 == 0 && ((reinterpret_cast<uintptr_t>(Al) | reinterpret_cast<uintptr_t>(x)) & 15u) == 0;
    const int n8 = vec ? n / 8 : 0;                    // groups of eight columns with 16-byte aligned rows
    const uint4 *a8 = reinterpret_cast<const uint4 *>(Al + (size_t)k * n);
    for (int g0 = tid; g0 < n8; g0 += 2 * 256) {
        const int g1 = g0 + 256;
        const uint4 av0 = __ldg(a8 + g0), av1 = g1 < n8 ? __ldg(a8 + g1) : make_uint4(0u, 0u, 0u, 0u);
        const uint32_t aw[8] = {av0.x, av0.y, av0.z, av0.w, av1.x, av1.y, av1.z, av1.w};
#pragma unroll
        for (int t = 0; t < kMaxTok; ++t) {
            if (t < M) {
                const uint4 *x8 = reinterpret_cast<const uint4 *>(x + (size_t)t * n);
                const uint4 xv0 = __ldg(x8 + g0), xv1 = g1 < n8 ? __ldg(x8 + g1) : make_uint4(0u, 0u, 0u, 0u);
                const uint32_t xw[8] = {xv0.x, xv0.y, xv0.z, xv0.w, xv1.x, xv1.y, xv1.z, xv1.w};
                float s = acc[t];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    s = fmaf(__uint_as_float(xw[e] << 16), __uint_as_float(aw[e] << 16), s);
                    s = fmaf(__uint_as_float(xw[e] & 0xFFFF0000u), __uint_as_float(aw[e] & 0xFFFF0000u), s);
                }
                acc[t] = s;
            }
        }
    }
    for (int j = 8 * n8 + tid; j < n; j += 256) {
        const float a = bf16f(Al[(size_t)k * n + j]);
#pragma unroll
        for (int t = 0; t < kMaxTok; ++t)
            if (t < M) acc[t] = fmaf(bf16f(x[(size_t)t * n + j]), a, acc[t]);
    }
#pragma unroll
    for (int t = 0; t < kMaxTok; ++t) {
        float v = acc[t];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        if (lane == 0) red[warp][t] = v;
    }
    __syncthreads();
    if (tid < M) {
        float v = 0.0f;
#pragma unroll
        for (int w = 0; w < 8; ++w) v += red[w][tid];
        u[(size_t)tid * r + k] = v;
    }
}

// y[t][i] = y32[t][i] + sum_k u[t][k] B_l[i][k], stored as bf16 (round to nearest even) or fp32.  A thread owns
// one row i for all tokens: its row of B_l is read once (16-byte loads when the rows are 16-byte multiples),
// u comes from shared memory.
constexpr int kAdapterRMax = 128;

__global__ void __launch_bounds__(128) lords_adapter_up_add_kernel(const float *__restrict__ y32, const float *__restrict__ u,
                                                                   const uint16_t *__restrict__ Bl, void *__restrict__ y, int y_f32,
                                                                   int M, int m, int r)
{
    __shared__ float us[kMaxTok][kAdapterRMax];
    for (int e = threadIdx.x; e < M * r; e += blockDim.x) us[e / r][e % r] = u[e];
    __syncthreads();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= m) return;
    float s[kMaxTok];
#pragma unroll
    for (int t = 0; t < kMaxTok; ++t) s[t] = 0.0f;
    const uint16_t *brow = Bl + (size_t)i * r;
    int k = 0;
    if (r % 8 == 0 && (reinterpret_cast<uintptr_t>(Bl) & 15u) == 0) {
        for (; k < r; k += 8) {
            const uint4 bv = __ldg(reinterpret_cast<const uint4 *>(brow + k));
            const uint32_t bw[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float b0 = __uint_as_float(bw[e] << 16), b1 = __uint_as_float(bw[e] & 0xFFFF0000u);
#pragma unroll
                for (int t = 0; t < kMaxTok; ++t)
                    if (t < M) s[t] = fmaf(us[t][k + 2 * e + 1], b1, fmaf(us[t][k + 2 * e], b0, s[t]));
            }
        }
    }
    for (; k < r; ++k) {
        const float b = bf16f(brow[k]);
#pragma unroll
        for (int t = 0; t < kMaxTok; ++t)
            if (t < M) s[t] = fmaf(us[t][k], b, s[t]);
    }
    float base[kMaxTok];
#pragma unroll
    for (int t = 0; t < kMaxTok; ++t) base[t] = t < M ? y32[(size_t)t * m + i] : 0.0f;     // all read before the first store
#pragma unroll
    for (int t = 0; t < kMaxTok; ++t) {
        if (t < M) {
            const float v = base[t] + s[t];
            if (y_f32) static_cast<float *>(y)[(size_t)t * m + i] = v;
            else static_cast<__nv_bfloat16 *>(y)[(size_t)t * m + i] = __float2bfloat16_rn(v);
        }
    }
}

}  // namespace

int launch_adapter(const uint16_t *x, const uint16_t *Al, const uint16_t *Bl, const float *y32, float *u, void *y, int y_f32,
                   int M, int m, int n, int r, cudaStream_t stream)
{
    if (M > kMaxTok || r > kAdapterRMax) return LORDS_ERR_UNSUPPORTED;
    // plain launches: as programmatic dependents (the next call's large CTAs then start early) the three kernels
    // of a call took 18.4 us instead of 16.5
    lords_adapter_down_kernel<<<(unsigned)r, 256, 0, stream>>>(x, Al, u, M, n, r);
    LORDS_CUDA_TRY(cudaGetLastError());
    lords_adapter_up_add_kernel<<<(unsigned)((m + 127) / 128), 128, 0, stream>>>(y32, u, Bl, y, y_f32, M, m, r);
    LORDS_CUDA_TRY(cudaGetLastError());
    return LORDS_OK;
}

}  // namespace lords
