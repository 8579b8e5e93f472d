// Host side of liblords.so: the C ABI of include/lords.h -- argument validation, the
// code packer, library state and the per-shape dispatch to the kernels.
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "lords_internal.h"

namespace lords {

State &state()
{
    static State s;
    return s;
}

// A small x in pinned host memory (mapped into the device's address space) is fetched by a kernel: a DMA copy
// of a few KB costs about 10 us in latency, a kernel's loads across the bus about 2 us.  The kernel is a
// programmatic dependent launch on both sides: it reads the host buffer (which no kernel writes) at once,
// waits for the previous kernel in the stream -- which may still be reading the staging buffer -- and only
// then stores; the forward kernel behind it may begin its set-up meanwhile.
constexpr size_t kDirectHostBytes = 1u << 20;   // above this the copy engines win
constexpr int kFetchBlocks = 64, kFetchThreads = 256;
constexpr int kFetchPerThread = (int)(kDirectHostBytes / 16 / (kFetchBlocks * kFetchThreads));   // 4

__global__ void __launch_bounds__(kFetchThreads) lords_fetch_host_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, size_t n16)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (size_t)gridDim.x * blockDim.x;
    uint4 v[kFetchPerThread];
#pragma unroll
    for (int k = 0; k < kFetchPerThread; ++k)
        if (t + k * stride < n16) v[k] = src[t + k * stride];
    asm volatile("griddepcontrol.wait;" ::: "memory");
#pragma unroll
    for (int k = 0; k < kFetchPerThread; ++k)
        if (t + k * stride < n16) dst[t + k * stride] = v[k];
}

// The device's address of a pinned, mapped host buffer; false for pageable or foreign memory.
static bool mapped_device_pointer(const void *host, void **dev)
{
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, host) != cudaSuccess) {
        (void)cudaGetLastError();
        return false;
    }
    if (a.type != cudaMemoryTypeHost || a.devicePointer == nullptr) return false;
    *dev = a.devicePointer;
    return true;
}

static int fetch_host(const void *src, void *dst, size_t bytes, cudaStream_t s)
{
    const size_t n16 = bytes / 16;      // bytes <= kDirectHostBytes: at most kFetchPerThread words per thread
    const size_t want = (n16 + kFetchThreads - 1) / kFetchThreads;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = cudaLaunchConfig_t{};
    cfg.gridDim = dim3((unsigned)(want < (size_t)kFetchBlocks ? (want > 0 ? want : 1) : (size_t)kFetchBlocks));
    cfg.blockDim = dim3(kFetchThreads);
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    LORDS_CUDA_TRY(cudaLaunchKernelEx(&cfg, lords_fetch_host_kernel, static_cast<const uint4 *>(src), static_cast<uint4 *>(dst), n16));
    return LORDS_OK;
}

int cuda_fail(cudaError_t e)
{
    state().last_cuda_error = (int)e;
    (void)cudaGetLastError();  // clear the sticky-free error so later calls start clean
    return LORDS_ERR_CUDA;
}

static int pack_group(int bits)
{
    switch (bits) {
        case 4: return 2;
        case 3: return 32;
        case 2: return 4;
        default: return 0;
    }
}

static int check_pack_shape(int64_t m, int64_t n, int bits)
{
    int g = pack_group(bits);
    if (g == 0) return LORDS_ERR_BITS;
    if (m < 0 || n < 0 || n % g != 0) return LORDS_ERR_SHAPE;
    return LORDS_OK;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int validate(const void *x, const uint8_t *q, const void *B, const void *A, const float *cb,
                    int bits, int M, int m, int n, int r, const void *y)
{
    if (!x || !q || !B || !A || !cb || !y) return LORDS_ERR_NULL;
    int g = pack_group(bits);
    if (g == 0) return LORDS_ERR_BITS;
    if (M < 1 || M > LORDS_M_MAX || m < 1 || n < 1 || r < 1 || r > LORDS_R_MAX) return LORDS_ERR_SHAPE;
    if (n % g != 0) return LORDS_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(q) || !aligned16(B) || !aligned16(A) || !aligned16(y)) return LORDS_ERR_ALIGN;
    if (!state().initialised) return LORDS_ERR_NOT_INIT;
    return LORDS_OK;
}

static int forward_common(const void *x, const uint8_t *q, const void *B, const void *A, const float *cb,
                          int bits, int M, int m, int n, int r, void *y, int y_f32, void *stream)
{
    int rc = validate(x, q, B, A, cb, bits, M, m, n, r, y);
    if (rc != LORDS_OK) return rc;
    State &st = state();
    Problem p;
    p.x = static_cast<const uint16_t *>(x);
    p.q = q;
    p.B = static_cast<const uint16_t *>(B);
    p.A = static_cast<const uint16_t *>(A);
    for (int c = 0; c < 16; ++c) p.levels[c] = c < (1 << bits) ? cb[c] : 0.0f;
    p.bits = bits; p.M = M; p.m = m; p.n = n; p.r = r;
    p.y = y; p.y_f32 = y_f32;
    st.last_launches = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    // Dispatch.  Each tensor-core path declines (LORDS_ERR_UNSUPPORTED) shapes outside its rules;
    // "auto" tries the decode kernels (M <= 2, then 3 <= M <= 16), then the scale-MMA kernel, then the
    // CUDA-core path.
    if (st.forced_path == 0 || st.forced_path == 2) {
        rc = launch_decode(p, st, s);
        if (rc != LORDS_ERR_UNSUPPORTED && rc != LORDS_ERR_WORKSPACE) return rc;
        if (st.forced_path == 2) return rc;
    }
    if (st.forced_path == 0 || st.forced_path == 4) {
        rc = launch_decode16(p, st, s);
        if (rc != LORDS_ERR_UNSUPPORTED && rc != LORDS_ERR_WORKSPACE) return rc;
        if (st.forced_path == 4) return rc;
    }
    if (st.forced_path == 0 || st.forced_path == 3) {
        rc = launch_umma(p, st, s);
        if (rc != LORDS_ERR_UNSUPPORTED && rc != LORDS_ERR_WORKSPACE) return rc;
        if (st.forced_path == 3) return rc;
    }
    return launch_simt(p, st, s);
}

}  // namespace lords

using namespace lords;

extern "C" {

int lords_version(void) { return LORDS_VERSION; }

const char *lords_strerror(int status)
{
    switch (status) {
        case LORDS_OK: return "ok";
        case LORDS_ERR_NULL: return "a required pointer is NULL";
        case LORDS_ERR_SHAPE: return "shape out of range or n not a multiple of the pack group";
        case LORDS_ERR_ALIGN: return "device pointer not 16-byte aligned";
        case LORDS_ERR_BITS: return "bits must be 2, 3 or 4";
        case LORDS_ERR_CODE_RANGE: return "code value >= 2^bits";
        case LORDS_ERR_NOT_INIT: return "lords_init has not been called";
        case LORDS_ERR_CUDA: return "CUDA call failed (see lords_last_cuda_error)";
        case LORDS_ERR_TIMEOUT: return "a bounded device-side wait timed out";
        case LORDS_ERR_WORKSPACE: return "scratch workspace too small for this problem";
        case LORDS_ERR_OPTION: return "unknown option or bad value";
        case LORDS_ERR_UNSUPPORTED: return "forced path does not support this shape";
        default: return "unknown status";
    }
}

int64_t lords_equivalent_rank(int64_t rows, int64_t cols, int64_t blk)
{
    if (rows < 1 || cols < 1 || blk < 1) return LORDS_ERR_SHAPE;
    // rows*cols < 2^63 for any realistic layer; guard the product anyway
    if (rows > (int64_t)3e9 || cols > (int64_t)3e9) return LORDS_ERR_SHAPE;
    return (rows * cols) / (blk * (rows + cols));
}

int64_t lords_packed_bytes(int64_t m, int64_t n, int bits)
{
    int rc = check_pack_shape(m, n, bits);
    if (rc != LORDS_OK) return rc;
    return m * (n * bits / 8);  // n * bits is a multiple of 8 for every pack group
}

int lords_pack_codes(const uint8_t *codes, int64_t m, int64_t n, int bits, uint8_t *packed)
{
    if (!codes || !packed) return LORDS_ERR_NULL;
    int rc = check_pack_shape(m, n, bits);
    if (rc != LORDS_OK) return rc;
    const int64_t row_bytes = lords_packed_bytes(1, n, bits);
    const unsigned limit = 1u << bits;
    for (int64_t i = 0; i < m; ++i) {
        const uint8_t *src = codes + i * n;
        uint8_t *dst = packed + i * row_bytes;
        // 64-bit shift register: codes enter at the top of the valid bits, whole bytes leave at the bottom
        uint64_t window = 0;
        int have = 0;
        for (int64_t j = 0; j < n; ++j) {
            unsigned c = src[j];
            if (c >= limit) return LORDS_ERR_CODE_RANGE;
            window |= (uint64_t)c << have;
            have += bits;
            while (have >= 8) {
                *dst++ = (uint8_t)window;
                window >>= 8;
                have -= 8;
            }
        }
    }
    return LORDS_OK;
}

int lords_unpack_codes(const uint8_t *packed, int64_t m, int64_t n, int bits, uint8_t *codes)
{
    if (!codes || !packed) return LORDS_ERR_NULL;
    int rc = check_pack_shape(m, n, bits);
    if (rc != LORDS_OK) return rc;
    const int64_t row_bytes = lords_packed_bytes(1, n, bits);
    const unsigned mask = (1u << bits) - 1u;
    for (int64_t i = 0; i < m; ++i) {
        const uint8_t *src = packed + i * row_bytes;
        uint8_t *dst = codes + i * n;
        uint64_t window = 0;
        int have = 0;
        for (int64_t j = 0; j < n; ++j) {
            if (have < bits) {
                window |= (uint64_t)(*src++) << have;
                have += 8;
            }
            dst[j] = (uint8_t)(window & mask);
            window >>= bits;
            have -= bits;
        }
    }
    return LORDS_OK;
}

int lords_init(int device, size_t workspace_bytes)
{
    State &st = state();
    if (st.initialised) lords_shutdown();
    int count = 0;
    LORDS_CUDA_TRY(cudaGetDeviceCount(&count));
    if (device < 0 || device >= count) return LORDS_ERR_SHAPE;
    LORDS_CUDA_TRY(cudaSetDevice(device));
    cudaDeviceProp prop;
    LORDS_CUDA_TRY(cudaGetDeviceProperties(&prop, device));
    st.device = device;
    st.sm_count = prop.multiProcessorCount;
    if (workspace_bytes == 0) workspace_bytes = (size_t)256 << 20;
    LORDS_CUDA_TRY(cudaMalloc(&st.workspace, workspace_bytes));
    st.workspace_bytes = workspace_bytes;
    st.counter_slots = 16384;
    const size_t small_bytes = 256 + sizeof(int) * (size_t)st.counter_slots;
    cudaError_t e = cudaMalloc(&st.status_word, small_bytes);
    if (e == cudaSuccess) e = cudaMemset(st.status_word, 0, small_bytes);
    st.counters = st.status_word + 64;
    if (e != cudaSuccess) {
        cudaFree(st.workspace);
        st.workspace = nullptr;
        return cuda_fail(e);
    }
    st.initialised = 1;
    return LORDS_OK;
}

int lords_shutdown(void)
{
    State &st = state();
    if (st.initialised) {
        cudaSetDevice(st.device);
        cudaDeviceSynchronize();
        cudaFree(st.workspace);
        cudaFree(st.status_word);
        if (st.stage_x) cudaFree(st.stage_x);
        if (st.stage_y) cudaFree(st.stage_y);
        if (st.bw_scratch) cudaFree(st.bw_scratch);
    }
    int fp = st.forced_path, fs = st.forced_splitk, fb = st.forced_bn;
    st = State();
    st.forced_path = fp;
    st.forced_splitk = fs;
    st.forced_bn = fb;
    return LORDS_OK;
}

int lords_linear_forward(const void *x, const uint8_t *Qpacked, const void *B, const void *A,
                         const float *codebook, int M, int m, int n, int r, void *y, void *stream)
{
    return forward_common(x, Qpacked, B, A, codebook, 4, M, m, n, r, y, 0, stream);
}

int lords_linear_forward_bits(const void *x, const uint8_t *Qpacked, const void *B, const void *A,
                              const float *codebook, int bits, int M, int m, int n, int r, void *y,
                              void *stream)
{
    return forward_common(x, Qpacked, B, A, codebook, bits, M, m, n, r, y, 0, stream);
}

int lords_linear_forward_f32(const void *x, const uint8_t *Qpacked, const void *B, const void *A,
                             const float *codebook, int bits, int M, int m, int n, int r, float *y32,
                             void *stream)
{
    return forward_common(x, Qpacked, B, A, codebook, bits, M, m, n, r, y32, 1, stream);
}

int lords_linear_forward_host(const void *x_host, const uint8_t *Qpacked, const void *B, const void *A,
                              const float *codebook, int bits, int M, int m, int n, int r, void *y_host,
                              void *stream)
{
    State &st = state();
    if (!x_host || !y_host) return LORDS_ERR_NULL;
    if (!st.initialised) return LORDS_ERR_NOT_INIT;
    if (M < 1 || M > LORDS_M_MAX || m < 1 || n < 1) return LORDS_ERR_SHAPE;
    const size_t xb = (size_t)M * n * 2, yb = (size_t)M * m * 2;
    if (xb > st.stage_x_bytes) {
        if (st.stage_x) cudaFree(st.stage_x);
        st.stage_x = nullptr; st.stage_x_bytes = 0;
        LORDS_CUDA_TRY(cudaMalloc(&st.stage_x, xb));
        st.stage_x_bytes = xb;
    }
    if (yb > st.stage_y_bytes) {
        if (st.stage_y) cudaFree(st.stage_y);
        st.stage_y = nullptr; st.stage_y_bytes = 0;
        LORDS_CUDA_TRY(cudaMalloc(&st.stage_y, yb));
        st.stage_y_bytes = yb;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    void *x_map = nullptr, *y_map = nullptr;
    const bool aligned = xb % 16 == 0 && yb % 16 == 0 && (reinterpret_cast<uintptr_t>(x_host) | reinterpret_cast<uintptr_t>(y_host)) % 16 == 0;
    const bool direct = aligned && xb <= kDirectHostBytes && yb <= kDirectHostBytes && mapped_device_pointer(x_host, &x_map) &&
                        mapped_device_pointer(y_host, &y_map);
    int rc;
    if (direct) {
        rc = fetch_host(x_map, st.stage_x, xb, s);
        if (rc != LORDS_OK) return rc;
    } else {
        LORDS_CUDA_TRY(cudaMemcpyAsync(st.stage_x, x_host, xb, cudaMemcpyHostToDevice, s));
    }
    // direct: the kernels store y straight into the mapped host buffer (no kernel reads y back), which saves the
    // copy-out launch
    rc = forward_common(st.stage_x, Qpacked, B, A, codebook, bits, M, m, n, r, direct ? y_map : st.stage_y, 0, stream);
    if (rc != LORDS_OK) return rc;
    if (direct) st.last_launches += 1;
    else LORDS_CUDA_TRY(cudaMemcpyAsync(y_host, st.stage_y, yb, cudaMemcpyDeviceToHost, s));
    return LORDS_OK;
}

int lords_quantize_codes(const void *W, const void *B, const void *A, const float *codebook, int bits, int m, int n,
                         int r, uint8_t *Qpacked, void *stream)
{
    if (!W || !B || !A || !codebook || !Qpacked) return LORDS_ERR_NULL;
    const int g = pack_group(bits);
    if (g == 0) return LORDS_ERR_BITS;
    if (m < 1 || n < 1 || r < 1 || r > LORDS_R_MAX || n % g != 0) return LORDS_ERR_SHAPE;
    if (!aligned16(W) || !aligned16(B) || !aligned16(A) || !aligned16(Qpacked)) return LORDS_ERR_ALIGN;
    State &st = state();
    if (!st.initialised) return LORDS_ERR_NOT_INIT;
    st.last_launches = 0;
    return launch_quantize(W, B, A, codebook, bits, m, n, r, Qpacked, st, static_cast<cudaStream_t>(stream));
}

int lords_transpose_codes(const uint8_t *Qpacked, int bits, int m, int n, uint8_t *Qt_packed, void *stream)
{
    if (!Qpacked || !Qt_packed) return LORDS_ERR_NULL;
    const int g = pack_group(bits);
    if (g == 0) return LORDS_ERR_BITS;
    if (m < 1 || n < 1 || n % g != 0 || m % g != 0) return LORDS_ERR_SHAPE;
    if (!aligned16(Qpacked) || !aligned16(Qt_packed)) return LORDS_ERR_ALIGN;
    State &st = state();
    if (!st.initialised) return LORDS_ERR_NOT_INIT;
    const int rc = launch_transpose_codes(Qpacked, m, n, bits, Qt_packed, static_cast<cudaStream_t>(stream));
    if (rc != LORDS_OK) return rc;
    st.last_launches = 1;
    st.last_path = "transpose_codes";
    return LORDS_OK;
}

// dx = g W^ is the forward of the transposed layer: W^T = L[Q^T] (.) (A^T B^T).
static int backward_input_common(const void *dy, const uint8_t *Qt, const void *B, const void *A, const float *cb, int bits,
                                 int M, int m, int n, int r, void *dx, int dx_f32, void *stream)
{
    if (!dy || !Qt || !B || !A || !cb || !dx) return LORDS_ERR_NULL;
    if (m < 1 || n < 1 || r < 1 || r > LORDS_R_MAX) return LORDS_ERR_SHAPE;
    if (!aligned16(B) || !aligned16(A)) return LORDS_ERR_ALIGN;
    State &st = state();
    if (!st.initialised) return LORDS_ERR_NOT_INIT;
    const size_t at_bytes = ((size_t)n * r * 2 + 255) & ~(size_t)255, bt_bytes = (size_t)r * m * 2;
    if (at_bytes + bt_bytes > st.bw_scratch_bytes) {
        if (st.bw_scratch) cudaFree(st.bw_scratch);
        st.bw_scratch = nullptr; st.bw_scratch_bytes = 0;
        LORDS_CUDA_TRY(cudaMalloc(&st.bw_scratch, at_bytes + bt_bytes));
        st.bw_scratch_bytes = at_bytes + bt_bytes;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint16_t *At = reinterpret_cast<uint16_t *>(st.bw_scratch), *Bt = reinterpret_cast<uint16_t *>(st.bw_scratch + at_bytes);
    // A [r][n] -> [n][r] and B [m][r] -> [r][m], one launch
    int rc = launch_transpose_bf16_pair(static_cast<const uint16_t *>(A), r, n, At, static_cast<const uint16_t *>(B), m, r, Bt, s);
    if (rc != LORDS_OK) return rc;
    // the transposed layer has n out-features and m in-features; its "B" is A^T and its "A" is B^T
    rc = forward_common(dy, Qt, At, Bt, cb, bits, M, n, m, r, dx, dx_f32, stream);
    if (rc != LORDS_OK) return rc;
    st.last_launches += 1;
    return LORDS_OK;
}

int lords_linear_backward_input(const void *dy, const uint8_t *Qt_packed, const void *B, const void *A, const float *codebook,
                                int bits, int M, int m, int n, int r, void *dx, void *stream)
{
    return backward_input_common(dy, Qt_packed, B, A, codebook, bits, M, m, n, r, dx, 0, stream);
}

int lords_linear_backward_input_f32(const void *dy, const uint8_t *Qt_packed, const void *B, const void *A,
                                    const float *codebook, int bits, int M, int m, int n, int r, float *dx32, void *stream)
{
    return backward_input_common(dy, Qt_packed, B, A, codebook, bits, M, m, n, r, dx32, 1, stream);
}

int lords_linear_backward_factors(const void *dy, const void *x, const uint8_t *Qpacked, const void *B, const void *A,
                                  const float *codebook, int bits, int M, int m, int n, int r, float *dB, float *dA,
                                  void *stream)
{
    if (!dy || !x || !Qpacked || !B || !A || !codebook || (!dB && !dA)) return LORDS_ERR_NULL;
    const int g = pack_group(bits);
    if (g == 0) return LORDS_ERR_BITS;
    if (M < 1 || M > LORDS_M_MAX || m < 1 || n < 1 || n % g != 0) return LORDS_ERR_SHAPE;
    if (r < 1 || r > LORDS_R_MAX) return LORDS_ERR_SHAPE;
    State &st = state();
    if (!st.initialised) return LORDS_ERR_NOT_INIT;
    return launch_backward_factors(static_cast<const uint16_t *>(dy), static_cast<const uint16_t *>(x), Qpacked,
                                   static_cast<const uint16_t *>(B), static_cast<const uint16_t *>(A), codebook, bits, M, m,
                                   n, r, dB, dA, st, static_cast<cudaStream_t>(stream));
}

int lords_linear_backward_qat(const void *dy, const void *x, const void *W, const uint8_t *Qpacked, const void *B, const void *A,
                              const float *codebook, int bits, int M, int m, int n, int r, float *dW, float *dB, float *dA,
                              void *stream)
{
    if (!dy || !x || !W || !Qpacked || !B || !A || !codebook || (!dW && !dB && !dA)) return LORDS_ERR_NULL;
    const int g = pack_group(bits);
    if (g == 0) return LORDS_ERR_BITS;
    if (M < 1 || M > LORDS_M_MAX || m < 1 || n < 1 || n % g != 0 || r < 1 || r > LORDS_R_MAX) return LORDS_ERR_SHAPE;
    if (!aligned16(dy) || !aligned16(x) || !aligned16(W) || (dW && !aligned16(dW))) return LORDS_ERR_ALIGN;
    State &st = state();
    if (!st.initialised) return LORDS_ERR_NOT_INIT;
    return launch_backward_qat(static_cast<const uint16_t *>(dy), static_cast<const uint16_t *>(x), static_cast<const uint16_t *>(W),
                               Qpacked, static_cast<const uint16_t *>(B), static_cast<const uint16_t *>(A), codebook, bits, M, m, n, r,
                               dW, dB, dA, st, static_cast<cudaStream_t>(stream));
}

static int blockscale_common(const void *x, const uint8_t *q, const void *scales, const float *cb, int bits, int blk, int M,
                             int m, int n, void *y, int y_f32, void *stream)
{
    if (!x || !q || !scales || !cb || !y) return LORDS_ERR_NULL;
    const int g = pack_group(bits);
    if (g == 0) return LORDS_ERR_BITS;
    if (M < 1 || m < 1 || n < 1 || n % g != 0 || blk < 1) return LORDS_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(q) || !aligned16(y)) return LORDS_ERR_ALIGN;
    State &st = state();
    if (!st.initialised) return LORDS_ERR_NOT_INIT;
    Problem p;
    p.x = static_cast<const uint16_t *>(x);
    p.q = q;
    p.B = nullptr; p.A = nullptr;
    for (int c = 0; c < 16; ++c) p.levels[c] = c < (1 << bits) ? cb[c] : 0.0f;
    p.bits = bits; p.M = M; p.m = m; p.n = n; p.r = 16;
    p.y = y; p.y_f32 = y_f32;
    st.last_launches = 0;
    return launch_blockscale16(p, static_cast<const uint16_t *>(scales), blk, st, static_cast<cudaStream_t>(stream));
}

int lords_blockscale_forward(const void *x, const uint8_t *Qpacked, const void *scales, const float *codebook, int bits,
                             int blk, int M, int m, int n, void *y, void *stream)
{
    return blockscale_common(x, Qpacked, scales, codebook, bits, blk, M, m, n, y, 0, stream);
}

int lords_blockscale_forward_f32(const void *x, const uint8_t *Qpacked, const void *scales, const float *codebook, int bits,
                                 int blk, int M, int m, int n, float *y32, void *stream)
{
    return blockscale_common(x, Qpacked, scales, codebook, bits, blk, M, m, n, y32, 1, stream);
}

static int adapter_common(const void *x, const uint8_t *q, const void *scales, const void *Al, const void *Bl, const float *cb,
                          int bits, int blk, int M, int m, int n, int r, void *y, int y_f32, void *stream)
{
    if (!Al || !Bl || !y) return LORDS_ERR_NULL;
    if (r < 1 || r > LORDS_R_MAX) return LORDS_ERR_SHAPE;
    State &st = state();
    if (!st.initialised) return LORDS_ERR_NOT_INIT;
    // scratch: the block-scaled product's fp32 accumulators [M][m], then u [M][r]
    const size_t y32_bytes = ((size_t)M * m * sizeof(float) + 255) & ~(size_t)255;
    if (M < 1 || m < 1 || y32_bytes + (size_t)M * r * sizeof(float) > st.workspace_bytes) return LORDS_ERR_WORKSPACE;
    float *y32 = reinterpret_cast<float *>(st.workspace), *u = reinterpret_cast<float *>(st.workspace + y32_bytes);
    int rc = blockscale_common(x, q, scales, cb, bits, blk, M, m, n, y32, 1, stream);
    if (rc != LORDS_OK) return rc;
    rc = launch_adapter(static_cast<const uint16_t *>(x), static_cast<const uint16_t *>(Al), static_cast<const uint16_t *>(Bl), y32, u,
                        y, y_f32, M, m, n, r, static_cast<cudaStream_t>(stream));
    if (rc != LORDS_OK) return rc;
    st.last_launches = 3;
    st.last_path = "blockscale16+adapter";
    return LORDS_OK;
}

int lords_adapter_forward(const void *x, const uint8_t *Qpacked, const void *scales, const void *A_l, const void *B_l,
                          const float *codebook, int bits, int blk, int M, int m, int n, int r, void *y, void *stream)
{
    return adapter_common(x, Qpacked, scales, A_l, B_l, codebook, bits, blk, M, m, n, r, y, 0, stream);
}

int lords_adapter_forward_f32(const void *x, const uint8_t *Qpacked, const void *scales, const void *A_l, const void *B_l,
                              const float *codebook, int bits, int blk, int M, int m, int n, int r, float *y32, void *stream)
{
    return adapter_common(x, Qpacked, scales, A_l, B_l, codebook, bits, blk, M, m, n, r, y32, 1, stream);
}

int lords_poll_status(void *stream)
{
    State &st = state();
    if (!st.initialised) return LORDS_ERR_NOT_INIT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    LORDS_CUDA_TRY(cudaStreamSynchronize(s));
    int word = 0;
    LORDS_CUDA_TRY(cudaMemcpy(&word, st.status_word, sizeof(int), cudaMemcpyDeviceToHost));
    if (word != 0) LORDS_CUDA_TRY(cudaMemset(st.status_word, 0, sizeof(int)));
    return word;
}

int lords_read_status_detail(uint64_t detail[2])
{
    State &st = state();
    if (!detail) return LORDS_ERR_NULL;
    if (!st.initialised) return LORDS_ERR_NOT_INIT;
    LORDS_CUDA_TRY(cudaDeviceSynchronize());
    LORDS_CUDA_TRY(cudaMemcpy(detail, st.status_word + 2, 2 * sizeof(uint64_t), cudaMemcpyDeviceToHost));
    LORDS_CUDA_TRY(cudaMemset(st.status_word + 2, 0, 2 * sizeof(uint64_t)));
    return LORDS_OK;
}

int lords_last_cuda_error(void) { return state().last_cuda_error; }

int lords_set_option(const char *key, const char *value)
{
    if (!key || !value) return LORDS_ERR_NULL;
    State &st = state();
    if (std::strcmp(key, "path") == 0) {
        if (std::strcmp(value, "auto") == 0) st.forced_path = 0;
        else if (std::strcmp(value, "simt") == 0) st.forced_path = 1;
        else if (std::strcmp(value, "decode") == 0) st.forced_path = 2;
        else if (std::strcmp(value, "umma") == 0 || std::strcmp(value, "prefill") == 0) st.forced_path = 3;
        else if (std::strcmp(value, "decode16") == 0) st.forced_path = 4;
        else return LORDS_ERR_OPTION;
        return LORDS_OK;
    }
    if (std::strcmp(key, "splitk") == 0) {
        char *end = nullptr;
        long v = std::strtol(value, &end, 10);
        if (end == value || *end != '\0' || v < 0 || v > 1024) return LORDS_ERR_OPTION;
        st.forced_splitk = (int)v;
        return LORDS_OK;
    }
    if (std::strcmp(key, "inject_status") == 0) {
        // test switch: write a value into the device status word, as a kernel that gave up would
        char *end = nullptr;
        long v = std::strtol(value, &end, 10);
        if (end == value || *end != '\0' || v < -64 || v > 0) return LORDS_ERR_OPTION;
        if (!st.initialised) return LORDS_ERR_NOT_INIT;
        const int word = (int)v;
        LORDS_CUDA_TRY(cudaMemcpy(st.status_word, &word, sizeof(int), cudaMemcpyHostToDevice));
        return LORDS_OK;
    }
    if (std::strcmp(key, "bn") == 0) {
        char *end = nullptr;
        long v = std::strtol(value, &end, 10);
        if (end == value || *end != '\0' || (v != 0 && v != 32 && v != 64 && v != 128 && v != 256)) return LORDS_ERR_OPTION;
        st.forced_bn = (int)v;
        return LORDS_OK;
    }
    return LORDS_ERR_OPTION;
}

const char *lords_last_path(void) { return state().last_path; }

int lords_last_launch_count(void) { return state().last_launches; }

}  // extern "C"
