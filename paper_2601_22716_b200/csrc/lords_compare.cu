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

// u[t][k] = sum_j x[t][j] A_l[k][j]: one block per adapter rank k, all tokens at once.
__global__ void __launch_bounds__(256) lords_adapter_down_kernel(const uint16_t *__restrict__ x, const uint16_t *__restrict__ Al,
                                                                 float *__restrict__ u, int M, int n, int r)
{
    __shared__ float red[8][kMaxTok];
    const int k = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float acc[kMaxTok];
#pragma unroll
    for (int t = 0; t < kMaxTok; ++t) acc[t] = 0.0f;
    for (int j = tid; j < n; j += 256) {
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

// y[t][i] = y32[t][i] + sum_k u[t][k] B_l[i][k], stored as bf16 (round to nearest even) or fp32.
__global__ void lords_adapter_up_add_kernel(const float *__restrict__ y32, const float *__restrict__ u,
                                            const uint16_t *__restrict__ Bl, void *__restrict__ y, int y_f32, int M, int m, int r)
{
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= (long long)M * m) return;
    const int t = (int)(e / m), i = (int)(e % m);
    float s = 0.0f;
    for (int k = 0; k < r; ++k) s = fmaf(u[(size_t)t * r + k], bf16f(Bl[(size_t)i * r + k]), s);
    const float v = y32[e] + s;
    if (y_f32) static_cast<float *>(y)[e] = v;
    else static_cast<__nv_bfloat16 *>(y)[e] = __float2bfloat16_rn(v);
}

}  // namespace

int launch_adapter(const uint16_t *x, const uint16_t *Al, const uint16_t *Bl, const float *y32, float *u, void *y, int y_f32,
                   int M, int m, int n, int r, cudaStream_t stream)
{
    if (M > kMaxTok) return LORDS_ERR_UNSUPPORTED;
    lords_adapter_down_kernel<<<(unsigned)r, 256, 0, stream>>>(x, Al, u, M, n, r);
    LORDS_CUDA_TRY(cudaGetLastError());
    const long long total = (long long)M * m;
    lords_adapter_up_add_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(y32, u, Bl, y, y_f32, M, m, r);
    LORDS_CUDA_TRY(cudaGetLastError());
    return LORDS_OK;
}

}  // namespace lords
