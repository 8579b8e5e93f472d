// Generic CUDA-core path: y = x (L[Q] (.) (BA))^T for any shape the interface accepts
// (any r <= LORDS_R_MAX, any M, bits 2/3/4, n only a multiple of the pack group).
// It is the fallback for shapes outside the tensor-core paths' tiling rules and the first
// path every other one is compared with.
//
// Work split: a CTA owns 32 output rows (4 warps x 8 rows), a tile of up to 8 tokens
// (grid.z) and a contiguous range of 128-column chunks (grid.y = split-K).  Per chunk the
// CTA stages A[:, chunk] and x[tile, chunk] in shared memory as fp32; a lane owns 4
// consecutive columns, rebuilds S = B A for its 8 rows x 4 columns in registers (Eq. 3),
// multiplies by the looked-up level (W^ = L[Q] (.) S) and accumulates x W^T in fp32.
// With split-K the partial sums go to scratch and a second kernel adds them in a fixed
// order, so results are bit-identical run to run.
#include <cuda_bf16.h>

#include "lords_internal.h"

namespace lords {

namespace {

constexpr int kRowsPerWarp = 8;
constexpr int kWarps = 4;
constexpr int kRowsPerCta = kRowsPerWarp * kWarps;  // 32
constexpr int kChunk = 128;                         // columns per staged chunk
constexpr int kTokTile = 8;

struct SimtParams {
    const uint16_t *x;
    const uint8_t *q;
    const uint16_t *B;
    const uint16_t *A;
    float levels[16];
    int bits, M, m, n, r;
    int chunks_per_split;   // 128-column chunks each grid.y slice walks
    int splits;
    float *partial;         // [splits][M][m] when splits > 1
    void *y;
    int y_f32;
};

__device__ __forceinline__ float bf16_bits_to_float(uint16_t h) { return __uint_as_float((uint32_t)h << 16); }

__device__ __forceinline__ void store_out(void *y, int y_f32, size_t idx, float v)
{
    if (y_f32) static_cast<float *>(y)[idx] = v;
    else static_cast<__nv_bfloat16 *>(y)[idx] = __float2bfloat16_rn(v);
}

__global__ void __launch_bounds__(kWarps * 32) lords_simt_kernel(const SimtParams p)
{
    extern __shared__ float smem[];
    float *sA = smem;                                // [r][kChunk]
    float *sX = sA + (size_t)p.r * kChunk;           // [kTokTile][kChunk]
    float *sB = sX + kTokTile * kChunk;              // [kRowsPerCta][r]
    __shared__ float sL[16];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row0 = blockIdx.x * kRowsPerCta;
    const int split = blockIdx.y;
    const int tok0 = blockIdx.z * kTokTile;
    const int ntok = min(kTokTile, p.M - tok0);
    const int64_t row_bytes = (int64_t)p.n * p.bits / 8;
    const unsigned mask = (1u << p.bits) - 1u;

    if (tid < 16) sL[tid] = p.levels[tid];
    for (int e = tid; e < kRowsPerCta * p.r; e += blockDim.x) {
        int rr = e / p.r, k = e - rr * p.r;
        int i = row0 + rr;
        sB[e] = i < p.m ? bf16_bits_to_float(p.B[(size_t)i * p.r + k]) : 0.0f;
    }

    float acc[kTokTile][kRowsPerWarp];
#pragma unroll
    for (int t = 0; t < kTokTile; ++t)
#pragma unroll
        for (int rr = 0; rr < kRowsPerWarp; ++rr) acc[t][rr] = 0.0f;

    const int nchunks = (p.n + kChunk - 1) / kChunk;
    const int c_begin = split * p.chunks_per_split;
    const int c_end = min(nchunks, c_begin + p.chunks_per_split);

    for (int c = c_begin; c < c_end; ++c) {
        const int j0 = c * kChunk;
        __syncthreads();  // previous chunk fully consumed (also orders the sB/sL fill)
        for (int e = tid; e < p.r * kChunk; e += blockDim.x) {
            int k = e / kChunk, jj = e - k * kChunk;
            int j = j0 + jj;
            sA[e] = j < p.n ? bf16_bits_to_float(p.A[(size_t)k * p.n + j]) : 0.0f;
        }
        for (int e = tid; e < kTokTile * kChunk; e += blockDim.x) {
            int t = e / kChunk, jj = e - t * kChunk;
            int j = j0 + jj;
            sX[e] = (t < ntok && j < p.n) ? bf16_bits_to_float(p.x[(size_t)(tok0 + t) * p.n + j]) : 0.0f;
        }
        __syncthreads();

        // S for 8 rows x 4 columns
        float s[kRowsPerWarp][4];
#pragma unroll
        for (int rr = 0; rr < kRowsPerWarp; ++rr) s[rr][0] = s[rr][1] = s[rr][2] = s[rr][3] = 0.0f;
        const float *bBase = sB + (warp * kRowsPerWarp) * p.r;
        for (int k = 0; k < p.r; ++k) {
            const float4 a = *reinterpret_cast<const float4 *>(sA + k * kChunk + lane * 4);
#pragma unroll
            for (int rr = 0; rr < kRowsPerWarp; ++rr) {
                const float b = bBase[rr * p.r + k];
                s[rr][0] = fmaf(b, a.x, s[rr][0]);
                s[rr][1] = fmaf(b, a.y, s[rr][1]);
                s[rr][2] = fmaf(b, a.z, s[rr][2]);
                s[rr][3] = fmaf(b, a.w, s[rr][3]);
            }
        }

        // codes of this lane's 4 columns for each of its rows -> W^ = L[Q] * S (kept in s)
        const int jl = j0 + lane * 4;
        const int64_t bit0 = (int64_t)jl * p.bits;
        const int64_t byte0 = bit0 >> 3;
        const int shift = (int)(bit0 & 7);
#pragma unroll
        for (int rr = 0; rr < kRowsPerWarp; ++rr) {
            const int i = row0 + warp * kRowsPerWarp + rr;
            uint32_t v = 0;
            if (i < p.m && jl < p.n) {
                const uint8_t *rowp = p.q + (size_t)i * row_bytes;
#pragma unroll
                for (int b = 0; b < 3; ++b)
                    if (byte0 + b < row_bytes) v |= (uint32_t)rowp[byte0 + b] << (8 * b);
            }
            v >>= shift;
#pragma unroll
            for (int qd = 0; qd < 4; ++qd) {
                const unsigned code = (v >> (qd * p.bits)) & mask;
                // columns beyond n carry zeros in sA/sX, so whatever code is read there adds 0
                s[rr][qd] *= sL[code];
            }
        }

#pragma unroll
        for (int t = 0; t < kTokTile; ++t) {
            if (t < ntok) {
                const float4 xv = *reinterpret_cast<const float4 *>(sX + t * kChunk + lane * 4);
#pragma unroll
                for (int rr = 0; rr < kRowsPerWarp; ++rr) {
                    float a = acc[t][rr];
                    a = fmaf(xv.x, s[rr][0], a);
                    a = fmaf(xv.y, s[rr][1], a);
                    a = fmaf(xv.z, s[rr][2], a);
                    a = fmaf(xv.w, s[rr][3], a);
                    acc[t][rr] = a;
                }
            }
        }
    }

    // fixed-order butterfly over the 32 lanes, then lane 0 stores
#pragma unroll
    for (int t = 0; t < kTokTile; ++t)
#pragma unroll
        for (int rr = 0; rr < kRowsPerWarp; ++rr) {
            float v = acc[t][rr];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
            acc[t][rr] = v;
        }
    if (lane == 0) {
#pragma unroll
        for (int t = 0; t < kTokTile; ++t) {
            if (t >= ntok) continue;
#pragma unroll
            for (int rr = 0; rr < kRowsPerWarp; ++rr) {
                const int i = row0 + warp * kRowsPerWarp + rr;
                if (i >= p.m) continue;
                const size_t o = (size_t)(tok0 + t) * p.m + i;
                if (p.splits > 1) p.partial[(size_t)split * p.M * p.m + o] = acc[t][rr];
                else store_out(p.y, p.y_f32, o, acc[t][rr]);
            }
        }
    }
}

// Sum split-K partials in index order and store (bf16 RNE or fp32).
__global__ void lords_splitk_reduce_kernel(const float *partial, int splits, size_t count, void *y, int y_f32)
{
    size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= count) return;
    float v = 0.0f;
    for (int s = 0; s < splits; ++s) v += partial[(size_t)s * count + e];
    store_out(y, y_f32, e, v);
}

}  // namespace

// The kernel's dynamic shared-memory limit is raised once per device, with that device current, to
// what the largest rank needs: both entry points that launch it then always find the same limit.
int simt_prepare_device(int dev)
{
    static bool done[64] = {};
    const int slot = dev >= 0 && dev < 64 ? dev : 0;
    if (!done[slot]) {
        const size_t most = ((size_t)LORDS_R_MAX * kChunk + kTokTile * kChunk + (size_t)kRowsPerCta * LORDS_R_MAX) * sizeof(float);
        LORDS_CUDA_TRY(cudaFuncSetAttribute(lords_simt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)most));
        done[slot] = true;
    }
    return LORDS_OK;
}

int launch_simt(const Problem &p, State &st, cudaStream_t stream)
{
    SimtParams k;
    k.x = p.x; k.q = p.q; k.B = p.B; k.A = p.A;
    for (int c = 0; c < 16; ++c) k.levels[c] = p.levels[c];
    k.bits = p.bits; k.M = p.M; k.m = p.m; k.n = p.n; k.r = p.r;
    k.y = p.y; k.y_f32 = p.y_f32;

    const int row_ctas = (p.m + kRowsPerCta - 1) / kRowsPerCta;
    const int tok_tiles = (p.M + kTokTile - 1) / kTokTile;
    const int nchunks = (p.n + kChunk - 1) / kChunk;
    int splits = st.forced_splitk;
    if (splits <= 0) {
        // aim for about four CTAs per SM, never finer than 4 chunks per split
        const long base = (long)row_ctas * tok_tiles;
        splits = (int)((4L * st.sm_count + base - 1) / base);
        if (splits > nchunks / 4) splits = nchunks / 4;
        if (splits < 1) splits = 1;
    }
    if (splits > nchunks) splits = nchunks;
    const size_t need = (size_t)splits * p.M * p.m * sizeof(float);
    if (splits > 1 && need > st.workspace_bytes) {
        splits = 1;  // scratch too small: run unsplit rather than fail
    }
    k.chunks_per_split = (nchunks + splits - 1) / splits;
    splits = (nchunks + k.chunks_per_split - 1) / k.chunks_per_split;
    k.splits = splits;
    k.partial = reinterpret_cast<float *>(st.workspace);

    const size_t smem = ((size_t)p.r * kChunk + kTokTile * kChunk + (size_t)kRowsPerCta * p.r) * sizeof(float);
    const int prc = simt_prepare_device(st.device);
    if (prc != LORDS_OK) return prc;
    dim3 grid(row_ctas, splits, tok_tiles);
    if (tok_tiles > 65535) return LORDS_ERR_SHAPE;
    lords_simt_kernel<<<grid, kWarps * 32, smem, stream>>>(k);
    LORDS_CUDA_TRY(cudaGetLastError());
    st.last_launches = 1;
    if (splits > 1) {
        const size_t count = (size_t)p.M * p.m;
        const int threads = 256;
        lords_splitk_reduce_kernel<<<(unsigned)((count + threads - 1) / threads), threads, 0, stream>>>(
            k.partial, splits, count, p.y, p.y_f32);
        LORDS_CUDA_TRY(cudaGetLastError());
        st.last_launches = 2;
    }
    st.last_path = "simt";
    return LORDS_OK;
}

}  // namespace lords

// ---------------------------------------------------------------------------------------------
// Allocation-free entry point.
//
// Some hosts of this library may not allocate device memory at all: a plugin loaded into an
// inference server that has already handed every byte of HBM to its own pool (cudaMalloc then
// fails or steals from that pool), or a latency-critical loop that cannot afford the implicit
// device-wide synchronisation cudaMalloc and cudaFree perform.  Such callers cannot use
// lords_init, whose job is to allocate the scratch workspace.  For them the split-K forward
// above is offered with its partial sums kept in a fixed array that is part of the loaded
// module image: every GPU that loads the library holds these 4 MiB until the process exits.
//
// In host code the array's name is only a stand-in for the device object, so its device address
// is looked up once per device with cudaGetSymbolAddress (that device being current) and that
// pointer is what the kernels receive.
// ---------------------------------------------------------------------------------------------
namespace lords {
namespace {

constexpr size_t kNoAllocFloats = LORDS_NOALLOC_MAX_FLOATS;
static __device__ __align__(256) float g_noalloc_partials[kNoAllocFloats];

constexpr int kMaxDevices = 64;
float *g_noalloc_ptr[kMaxDevices] = {};   // device address of g_noalloc_partials, per device
int g_noalloc_sms[kMaxDevices] = {};

}  // namespace
}  // namespace lords

extern "C" int lords_linear_forward_noalloc(const void *x, const uint8_t *Qpacked, const void *B, const void *A,
                                            const float *codebook, int bits, int M, int m, int n, int r,
                                            void *y, void *stream)
{
    using namespace lords;
    if (!x || !Qpacked || !B || !A || !codebook || !y) return LORDS_ERR_NULL;
    if (bits != 2 && bits != 3 && bits != 4) return LORDS_ERR_BITS;
    const int group = bits == 4 ? 2 : (bits == 3 ? 32 : 4);
    if (M < 1 || M > LORDS_M_MAX || m < 1 || n < 1 || r < 1 || r > LORDS_R_MAX || n % group != 0)
        return LORDS_ERR_SHAPE;
    const uintptr_t all = (uintptr_t)x | (uintptr_t)Qpacked | (uintptr_t)B | (uintptr_t)A | (uintptr_t)y;
    if (all & 15u) return LORDS_ERR_ALIGN;
    // two partial copies of the output are the least this variant needs
    if (2 * (size_t)M * (size_t)m > kNoAllocFloats) return LORDS_ERR_WORKSPACE;

    int dev = -1;
    LORDS_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return LORDS_ERR_SHAPE;
    if (g_noalloc_ptr[dev] == nullptr) {
        // one-time set-up for this device (it is the current one): resolve the array's device address
        float *ptr = nullptr;
        LORDS_CUDA_TRY(cudaGetSymbolAddress((void **)&ptr, g_noalloc_partials));
        int sms = 0;
        LORDS_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        g_noalloc_sms[dev] = sms;
        g_noalloc_ptr[dev] = ptr;
    }

    SimtParams k;
    k.x = static_cast<const uint16_t *>(x); k.q = Qpacked;
    k.B = static_cast<const uint16_t *>(B); k.A = static_cast<const uint16_t *>(A);
    for (int c = 0; c < 16; ++c) k.levels[c] = c < (1 << bits) ? codebook[c] : 0.0f;
    k.bits = bits; k.M = M; k.m = m; k.n = n; k.r = r;
    k.y = y; k.y_f32 = 0;

    const int row_ctas = (m + kRowsPerCta - 1) / kRowsPerCta;
    const int tok_tiles = (M + kTokTile - 1) / kTokTile;
    if (tok_tiles > 65535) return LORDS_ERR_SHAPE;
    const int nchunks = (n + kChunk - 1) / kChunk;
    const long base = (long)row_ctas * tok_tiles;
    int splits = (int)((4L * g_noalloc_sms[dev] + base - 1) / base);
    if (splits > nchunks / 4) splits = nchunks / 4;
    const size_t fit = kNoAllocFloats / ((size_t)M * m);      // >= 2, checked above
    if ((size_t)splits > fit) splits = (int)fit;
    if (splits < 2) splits = 2;                               // always the scratch-using variant
    if (splits > nchunks) splits = nchunks;                   // a single chunk: one split, via scratch all the same
    k.chunks_per_split = (nchunks + splits - 1) / splits;
    splits = (nchunks + k.chunks_per_split - 1) / k.chunks_per_split;
    k.splits = splits;
    k.partial = g_noalloc_ptr[dev];

    const size_t smem = ((size_t)r * kChunk + kTokTile * kChunk + (size_t)kRowsPerCta * r) * sizeof(float);
    const int prc = simt_prepare_device(dev);
    if (prc != LORDS_OK) return prc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (splits > 1) {
        lords_simt_kernel<<<dim3(row_ctas, splits, tok_tiles), kWarps * 32, smem, s>>>(k);
        LORDS_CUDA_TRY(cudaGetLastError());
        const size_t count = (size_t)M * m;
        lords_splitk_reduce_kernel<<<(unsigned)((count + 255) / 256), 256, 0, s>>>(k.partial, splits, count, y, 0);
        LORDS_CUDA_TRY(cudaGetLastError());
    } else {
        // n fits one chunk: the lone split still lands in the static array, then is rounded out of it
        k.splits = 2;  // makes the kernel take its "write partials" branch; slice 1 is never produced
        k.chunks_per_split = nchunks;
        lords_simt_kernel<<<dim3(row_ctas, 1, tok_tiles), kWarps * 32, smem, s>>>(k);
        LORDS_CUDA_TRY(cudaGetLastError());
        const size_t count = (size_t)M * m;
        lords_splitk_reduce_kernel<<<(unsigned)((count + 255) / 256), 256, 0, s>>>(k.partial, 1, count, y, 0);
        LORDS_CUDA_TRY(cudaGetLastError());
    }
    return LORDS_OK;
}
