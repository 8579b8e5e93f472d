/*
 * lords.h -- C ABI of the B200 (sm_100a) LoRDS dequantize-and-multiply library.
 *
 * The library computes one quantised linear layer of LoRDS inference:
 *
 *     y = x * ( L[Q] (.) (B A) )^T
 *
 *   x : M x n activations (tokens x in-features)
 *   Q : m x n codes, bits per code 2, 3 or 4, packed (layout below)
 *   L : level table with 2^bits entries (the target data type's discrete levels,
 *       e.g. NF4; Sec. 3.1 "Round(.) ... nearest discrete levels of a target data type")
 *   B : m x r, A : r x n -- the low-rank factors of the element-wise scale matrix
 *       S = B A (Sec. 3.2, Eq. 3); S is rebuilt on chip and never stored in full
 *   y : M x m outputs (tokens x out-features)
 *
 * The dequantised weight is W^ = Q (.) (BA) with Q_ij a level of L (Sec. 3.2-3.3,
 * Alg. 1 step 2.1; Eq. 2 is its block-wise special case), and the layer is
 * y = x W^T with W stored out-features x in-features (Table 7 lists shapes that way).
 * Note the paper writes W in R^{n x m}; this interface uses m for out-features and
 * n for in-features (the reduction axis).
 *
 * Around that layer the library also has, each documented at its declaration: the quantisation
 * step that produces the codes (Alg. 1 step 2.1), the layer's backward for multiplicative
 * fine-tuning of B and A (Sec. 3.4) and for quantisation-aware training (Eq. 4-5), and two
 * comparators for the paper's efficiency table (a block-scaled layer, Eq. 2, and that layer with an
 * additive adapter).
 *
 * Conventions
 *   - every function returns an int status: LORDS_OK (0) or a negative LORDS_ERR_*;
 *     nothing throws, exits or traps.  Size-returning calls return a negative
 *     LORDS_ERR_* on error.
 *   - "device" pointers are CUDA global-memory pointers on the device given to
 *     lords_init; "host" pointers are ordinary CPU memory.
 *   - all matrices are dense row-major without padding.  x, B, A, y hold bf16
 *     (IEEE bfloat16 bit patterns, 2 bytes); device pointers must be 16-byte aligned.
 *   - the caller owns every buffer it passes for the whole asynchronous lifetime of
 *     the call; the library neither retains nor frees them.  x/y aliasing is undefined.
 *   - the tensor-core kernels are launched with programmatic dependent launch: they may begin while
 *     the previous kernel on `stream` is still draining, and until that kernel has finished they
 *     read only the weights (Qpacked, B, A); x is read, and y written, after it.  So the weights must
 *     not be produced by work that is still in flight on `stream` when a forward call is made
 *     (synchronise the stream once after loading or updating weights); activations may be.
 *   - precision and range: products are accumulated in fp32.  The tensor-core kernels hold their
 *     operands in fp16, each rounded once: the dequantised weight L[Q_ij] * (BA)_ij (M > 2), or the bare
 *     level L[Q_ij] and the product A_kj * x_tj (M <= 2), and x itself (M > 2).  These values must lie
 *     within fp16's range: magnitudes above 65504 overflow to infinity, magnitudes below 6.1e-5 are
 *     rounded to multiples of 6e-8 (which matters only where such terms dominate a sum).  Layer
 *     weights and activations of the usual scales (|x| up to a few thousand, factors around 1e-2 to 1)
 *     are far inside; the CUDA-core path ("path" = "simt") is fp32 throughout and has no such limit.
 *   - forward calls validate on the host, enqueue work on `stream` and return
 *     without synchronising.  They use library-owned scratch memory, so two forward
 *     calls may only overlap on the GPU if they are ordered on the same stream.
 *
 * Packed code layout (the paper does not fix one; this is the library's definition)
 *   rows are packed independently; row i starts at byte i * n * bits / 8 and is a
 *   little-endian bit stream with code j at bit offset j * bits:
 *     bits = 4 : byte b = code[2b] | code[2b+1] << 4            (n % 2  == 0)
 *     bits = 3 : 32 codes -> 96-bit little-endian integer, 12 B  (n % 32 == 0)
 *     bits = 2 : byte b = code[4b+q] << 2q, q = 0..3             (n % 4  == 0)
 *   Code c selects level L[c].
 */
#ifndef LORDS_H_
#define LORDS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LORDS_VERSION 100 /* major*10000 + minor*100 + patch */

/* status codes */
#define LORDS_OK 0
#define LORDS_ERR_NULL (-1)        /* a required pointer is NULL */
#define LORDS_ERR_SHAPE (-2)       /* M, m, n or r out of range, or n not a multiple of the pack group */
#define LORDS_ERR_ALIGN (-3)       /* a device pointer is not 16-byte aligned */
#define LORDS_ERR_BITS (-4)        /* bits is not 2, 3 or 4 */
#define LORDS_ERR_CODE_RANGE (-5)  /* a code is >= 2^bits */
#define LORDS_ERR_NOT_INIT (-6)    /* lords_init has not been called (or failed) */
#define LORDS_ERR_CUDA (-7)        /* a CUDA runtime/driver call failed; see lords_last_cuda_error */
#define LORDS_ERR_TIMEOUT (-8)     /* a bounded device-side wait gave up (reported by lords_poll_status) */
#define LORDS_ERR_WORKSPACE (-9)   /* the problem needs more scratch memory than lords_init reserved */
#define LORDS_ERR_OPTION (-10)     /* unknown option key or bad value */
#define LORDS_ERR_UNSUPPORTED (-11)/* the forced path cannot run this shape */

#define LORDS_R_MAX 128            /* largest supported rank r */
#define LORDS_M_MAX 65536          /* largest supported token count M */

/* Library version (LORDS_VERSION of the built library). */
int lords_version(void);

/* Static, human-readable text for a status code.  Never NULL. */
const char *lords_strerror(int status);

/*
 * Equivalent-rank rule of Sec. 3.2 / App. A: r = floor(rows*cols / (blk*(rows+cols))), the rank
 * whose factor parameters r*(rows+cols) fit the block-wise scale budget rows*cols/blk.
 * Returns the rank (>= 0) or LORDS_ERR_SHAPE.
 */
int64_t lords_equivalent_rank(int64_t rows, int64_t cols, int64_t blk);

/* Bytes of the packed form of an m x n code matrix: m * n * bits / 8, or a negative status. */
int64_t lords_packed_bytes(int64_t m, int64_t n, int bits);

/*
 * Pack codes (offline, once per layer; the storage implied by the paper's "4-bit" accounting).
 *   codes  : host, m*n bytes, one code per byte, row-major
 *   packed : host, lords_packed_bytes(m, n, bits) bytes, fully overwritten
 * Pure CPU, deterministic.  Fails with LORDS_ERR_CODE_RANGE (packed contents then unspecified)
 * if any code >= 2^bits.
 */
int lords_pack_codes(const uint8_t *codes, int64_t m, int64_t n, int bits, uint8_t *packed);

/* Inverse of lords_pack_codes: packed (host) -> codes (host, m*n bytes). */
int lords_unpack_codes(const uint8_t *packed, int64_t m, int64_t n, int bits, uint8_t *codes);

/*
 * Bind the library to CUDA device `device` and allocate its scratch memory (split-K
 * partial sums, converted activations, a device status word).  workspace_bytes = 0 selects
 * the default (256 MiB).  Calling it again re-initialises.  Must precede any forward call.
 */
int lords_init(int device, size_t workspace_bytes);

/* Free everything lords_init allocated.  Safe to call when not initialised. */
int lords_shutdown(void);

/*
 * The fused dequantize-and-multiply y = x (L[Q] (.) (BA))^T for 4-bit codes (Sec. 3.2-3.4;
 * the operator timed in Sec. 4.4).
 *   x        : device, bf16 [M][n]
 *   Qpacked  : device, packed 4-bit codes, m * n / 2 bytes
 *   B        : device, bf16 [m][r]
 *   A        : device, bf16 [r][n]
 *   codebook : HOST, 16 floats, level table L (copied into the launch; may be freed on return)
 *   y        : device, bf16 [M][m]; accumulation is fp32, the store rounds to nearest even
 *   stream   : a cudaStream_t passed as void* (NULL = the default stream)
 * Ranges: 1 <= M <= LORDS_M_MAX, 1 <= r <= LORDS_R_MAX, m >= 1, n >= 2 and even.
 */
int lords_linear_forward(const void *x, const uint8_t *Qpacked, const void *B, const void *A,
                         const float *codebook, int M, int m, int n, int r, void *y, void *stream);

/* Same with an explicit code width: bits in {2, 3, 4}; codebook holds 2^bits floats. */
int lords_linear_forward_bits(const void *x, const uint8_t *Qpacked, const void *B, const void *A,
                              const float *codebook, int bits, int M, int m, int n, int r, void *y,
                              void *stream);

/*
 * Verification entry: identical kernels, but the epilogue stores the fp32 accumulator.
 *   y32 : device, float [M][m]
 */
int lords_linear_forward_f32(const void *x, const uint8_t *Qpacked, const void *B, const void *A,
                             const float *codebook, int bits, int M, int m, int n, int r, float *y32,
                             void *stream);

/*
 * End-to-end variant for callers whose activations live in host memory: x_host (bf16 [M][n])
 * and y_host (bf16 [M][m]) are HOST pointers (pinned memory recommended, otherwise the copies
 * are synchronous); the weights Qpacked, B, A stay device-resident as above.  Enqueues, on
 * `stream`, the host-to-device copy of x, the same kernels as lords_linear_forward_bits and
 * the device-to-host copy of y, and returns without synchronising.  With buffers of up to 1 MiB
 * in pinned (mapped) host memory no DMA copy is made: a small kernel reads x from the host memory
 * (it may do so while the previous kernel in the stream is still running: x_host must not be the
 * target of work enqueued earlier on the stream) and the forward kernels store y straight into
 * y_host, which saves most of the latency of two DMA copies; larger or pageable buffers go through
 * cudaMemcpyAsync.  The device staging
 * buffers are library-owned and grow (cudaMalloc) the first time a larger M*n or M*m is seen,
 * so the first call of a given size must not be made during stream capture.
 */
int lords_linear_forward_host(const void *x_host, const uint8_t *Qpacked, const void *B, const void *A,
                              const float *codebook, int bits, int M, int m, int n, int r, void *y_host,
                              void *stream);

/*
 * Quantisation step of the alternating refinement (Alg. 1, step 2.1; Sec. 3.3): with the factors fixed,
 *     Q_ij = argmin over the codes c of (S_ij * L[c] - W_ij)^2,   S = B A (Eq. 3),
 * written as packed codes in the layout above (ready for the forward calls).  The paper does not say
 * which level wins a tie: the lowest code does.  S is accumulated in fp32 and every level is tried in
 * fp32, so a weight within rounding distance of the midpoint between two levels' products may get
 * either neighbour.
 *   W        : device, bf16 [m][n], the weight to quantise (out-features x in-features)
 *   B, A     : device, bf16 [m][r] and [r][n]
 *   codebook : HOST, 2^bits floats (ascending or not: codes index it as given)
 *   Qpacked  : device, lords_packed_bytes(m, n, bits) bytes, fully overwritten
 * Ranges as for the forward calls (n a multiple of the pack group); needs lords_init; enqueues on
 * `stream` and returns without synchronising.
 */
int lords_quantize_codes(const void *W, const void *B, const void *A, const float *codebook, int bits, int m, int n,
                         int r, uint8_t *Qpacked, void *stream);

/*
 * Backward of the layer with the codes fixed: what multiplicative fine-tuning of B and A needs
 * (Sec. 3.4; the chain rule through S = BA is that of Eq. 5).  With g = dL/dy, bf16 [M][m]:
 *     dx = g W^  [M][n],     dS = (g^T x) (.) L[Q]  (never stored),     dB = dS A^T  [m][r],     dA = B^T dS  [r][n].
 *
 * lords_transpose_codes: Qt_packed (device, lords_packed_bytes(n, m, bits) bytes) receives the packed
 *   codes of Q^T, n rows of m codes; m must be a multiple of the pack group like n.  The codes are
 *   frozen during fine-tuning, so this is done once per layer.
 * lords_linear_backward_input[_f32]: dx = g W^ as the forward of the transposed layer,
 *   W^T = L[Q^T] (.) (A^T B^T): the same kernels, dispatch, operand ranges and error behaviour as the
 *   forward calls, with (m, n) exchanged.  B and A are the layer's own factors ([m][r], [r][n]); their
 *   transposes are made per call in library-owned scratch that grows (cudaMalloc) when a larger layer
 *   is seen, so the first call of a given size must not be made during stream capture.
 *   dx: device, bf16 [M][n] (or float [M][n] for _f32).
 * lords_linear_backward_factors: dB (device, float [m][r]) and dA (device, float [r][n]); either may
 *   be NULL.  The product g^T x is formed tile by tile on the tensor cores (bf16 operands as given,
 *   fp32 accumulation) when m and n are multiples of 8, else on the CUDA cores; the level multiply
 *   and the contractions with A and B are fp32 on the CUDA cores.  Every element is summed in a
 *   fixed order (runs are bit-identical).  The tiles' contributions go through the lords_init
 *   workspace; without room there a slower schedule without scratch memory runs.
 *   x: device, bf16 [M][n].  Any bits in {2,3,4}, r <= LORDS_R_MAX.
 * All enqueue on `stream` and return without synchronising; all need lords_init.
 */
int lords_transpose_codes(const uint8_t *Qpacked, int bits, int m, int n, uint8_t *Qt_packed, void *stream);
int lords_linear_backward_input(const void *dy, const uint8_t *Qt_packed, const void *B, const void *A, const float *codebook,
                                int bits, int M, int m, int n, int r, void *dx, void *stream);
int lords_linear_backward_input_f32(const void *dy, const uint8_t *Qt_packed, const void *B, const void *A,
                                    const float *codebook, int bits, int M, int m, int n, int r, float *dx32, void *stream);
int lords_linear_backward_factors(const void *dy, const void *x, const uint8_t *Qpacked, const void *B, const void *A,
                                  const float *codebook, int bits, int M, int m, int n, int r, float *dB, float *dA,
                                  void *stream);

/*
 * Gradients of quantisation-aware training with the straight-through estimator (Sec. 3.3, Eq. 4-5):
 * the fake-quantised weight is W^ = Round(W (/) S) (.) S, S = B A, the codes are those of the current
 * rounding (lords_quantize_codes), and with g = dL/dy
 *     dL/dW = dL/dW^ = g^T x                              (Eq. 4),
 *     dL/dS = dL/dW^ (.) (L[Q] - W (/) S)                  (Eq. 5; 0 where S is exactly 0),
 *     dB = dL/dS A^T,   dA = B^T dL/dS.
 *   W  : device, bf16 [m][n], the latent full-precision weight
 *   dW : device, float [m][n] or NULL;  dB : device, float [m][r] or NULL;  dA : device, float [r][n] or NULL
 * Runs on the tensor-core schedule of lords_linear_backward_factors when m and n are multiples of 8
 * and the lords_init workspace has room for the tiles' contributions; otherwise on the CUDA cores,
 * one pass over W per requested factor gradient, without scratch memory (any shape the forward calls
 * accept).  The quotient is formed in fp32 (on the tensor-core schedule by a reciprocal with one residual
 * correction: exact when W / S is representable, else within a rounding error or two; a non-zero |S| below
 * the smallest normal float, 1.2e-38, is outside the supported range there); S is accumulated in fp32 from the exact products of the
 * bf16 factors (by a tensor-core scale MMA when r is a multiple of 8 up to 64 on the tensor-core
 * schedule, else in ascending order of the rank).  An output that is NULL is not touched.  Enqueues on `stream` and returns without
 * synchronising.
 */
int lords_linear_backward_qat(const void *dy, const void *x, const void *W, const uint8_t *Qpacked, const void *B, const void *A,
                              const float *codebook, int bits, int M, int m, int n, int r, float *dW, float *dB, float *dA,
                              void *stream);

/*
 * Comparators for the paper's efficiency claims (Sec. 4.4, Table 6), on the same GPU and the same packed
 * codes: a block-scaled layer (Eq. 2), and that layer with an additive low-rank adapter that cannot be
 * merged into the quantised weights (Sec. 3.4).
 *     lords_blockscale_forward:  y = x (L[Q] (.) (s (x) 1))^T,  scales: device, bf16 [m][ceil(n / blk)],
 *         one scale per row and block of `blk` consecutive in-feature columns (blk a multiple of 64).
 *     lords_adapter_forward:     y = x W_block^T + (x A_l^T) B_l^T,  A_l: device, bf16 [r][n];
 *         B_l: device, bf16 [m][r]; three launches (the block-scaled product into the library's
 *         workspace in fp32, u = x A_l^T, y = product + u B_l^T).
 * M <= 16 (they are decode comparators); n a multiple of 64 (2- and 4-bit codes) or 128 (3-bit); other
 * shapes return LORDS_ERR_UNSUPPORTED.  y: device, bf16 [M][m] (float for the _f32 variants).  Operand
 * ranges, status word and error behaviour as for the forward calls.
 */
int lords_blockscale_forward(const void *x, const uint8_t *Qpacked, const void *scales, const float *codebook, int bits,
                             int blk, int M, int m, int n, void *y, void *stream);
int lords_blockscale_forward_f32(const void *x, const uint8_t *Qpacked, const void *scales, const float *codebook, int bits,
                                 int blk, int M, int m, int n, float *y32, void *stream);
int lords_adapter_forward(const void *x, const uint8_t *Qpacked, const void *scales, const void *A_l, const void *B_l,
                          const float *codebook, int bits, int blk, int M, int m, int n, int r, void *y, void *stream);
int lords_adapter_forward_f32(const void *x, const uint8_t *Qpacked, const void *scales, const void *A_l, const void *B_l,
                              const float *codebook, int bits, int blk, int M, int m, int n, int r, float *y32, void *stream);

/*
 * Allocation-free forward (the paper has no counterpart: this is a deployment convenience).
 * For callers that must not allocate device memory -- for instance a plugin inside a server
 * whose memory pool already owns all of HBM, or a latency-critical loop that cannot take the
 * device-wide synchronisation cudaMalloc/cudaFree imply.  Same arguments and result as
 * lords_linear_forward_bits (device pointers, host codebook, bf16 y), but it needs no
 * lords_init and calls no allocator: it runs the split-K CUDA-core kernels with their partial
 * sums in a fixed LORDS_NOALLOC_MAX_FLOATS-float (4 MiB) array inside the library image, which
 * every GPU that loads the library holds until the process exits.
 *   - limit: 2 * M * m <= LORDS_NOALLOC_MAX_FLOATS, otherwise LORDS_ERR_WORKSPACE;
 *   - it works on the calling thread's current CUDA device; the first call on each device also
 *     resolves the array's device address, so make that first call outside any stream capture;
 *   - all calls share the one array: every slot a call reads it has written itself, so stale
 *     contents are harmless, but two calls that overlap on the GPU (different streams) race --
 *     order them on one stream.
 */
#define LORDS_NOALLOC_MAX_FLOATS (1u << 20)
int lords_linear_forward_noalloc(const void *x, const uint8_t *Qpacked, const void *B, const void *A,
                                 const float *codebook, int bits, int M, int m, int n, int r, void *y,
                                 void *stream);

/*
 * Read and clear the device status word.  Synchronises `stream` first.  Returns LORDS_OK, or
 * the error a kernel recorded (LORDS_ERR_TIMEOUT when a bounded wait ran out).
 * Every device-side wait of the tensor-core kernels is bounded (50 ms); a wait that runs out records
 * LORDS_ERR_TIMEOUT here, every other wait then ends at once, and the kernels finish without
 * writing their results.  Forward calls do not report this themselves: when this call returns
 * non-zero, the y of every forward call since the previous poll is undefined, and so is the y of
 * calls made before the word is cleared by this call.
 */
int lords_poll_status(void *stream);

/*
 * Diagnosis of LORDS_ERR_TIMEOUT: reads and clears the record that the first device-side wait to run
 * out left behind (host pointer to two 64-bit words; both zero if none ran out).
 *   detail[0]: bit 63 set; bits 0..7 a tag naming the wait inside its kernel, bit 8 the phase parity
 *              waited for, bits 16..23 the warp, bits 32..62 the CTA (blockIdx.x)
 *   detail[1]: bits 0..31 the shared-memory address of the barrier, bits 32..63 how many rounds of
 *              64 tries the wait made
 * Synchronises the device.
 */
int lords_read_status_detail(uint64_t detail[2]);

/* The cudaError_t (as int) of the most recent failed CUDA call, 0 if none. */
int lords_last_cuda_error(void);

/*
 * Measurement switches.  Keys: "path" = "auto" | "simt" | "decode" (reassociated-form kernel,
 * M <= 2) | "decode16" (scale-MMA form with 128-column k-steps, 3 <= M <= 16) | "umma" (scale-MMA
 * kernel for any M; "prefill" is an alias);
 * "splitk" = "0" (auto) or a positive integer (CTAs sharing one tile's k-range); "bn" = "0" (auto)
 * or the token tile 32, 64, 128, 256 of the scale-MMA kernel for M > 16; "inject_status" = "0" or a
 * negative status code: writes that value into the device status word, as a kernel that gave up would
 * (a test switch).  Unknown keys: LORDS_ERR_OPTION.
 */
int lords_set_option(const char *key, const char *value);

/* Name of the path the most recent call dispatched to ("simt", "decode", "decode16", "umma"; "quantize",
 * "quantize_simt" for lords_quantize_codes). */
const char *lords_last_path(void);

/* Number of kernels the most recent forward call launched. */
int lords_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* LORDS_H_ */
