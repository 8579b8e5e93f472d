// Internal declarations shared by the translation units of liblords.so (not installed).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "lords.h"

namespace lords {

// One forward call, validated.  Pointers are device pointers except the level table,
// which travels by value inside the kernel parameters.
struct Problem {
    const uint16_t *x;   // bf16 [M][n]
    const uint8_t *q;    // packed codes, m * n * bits / 8 bytes
    const uint16_t *B;   // bf16 [m][r]
    const uint16_t *A;   // bf16 [r][n]
    float levels[16];    // L, 2^bits entries used
    int bits, M, m, n, r;
    void *y;             // bf16 [M][m] or float [M][m]
    int y_f32;           // 1: store the fp32 accumulator
};

// Library-owned device memory and switches (one instance per process).
struct State {
    int initialised = 0;
    int device = -1;
    int sm_count = 0;
    uint8_t *workspace = nullptr;   // scratch: split-K partials / converted activations
    size_t workspace_bytes = 0;
    int *status_word = nullptr;     // device int, 0 = OK, else a LORDS_ERR_* a kernel recorded
    int *counters = nullptr;        // split-K arrival counters, zero between calls
    int counter_slots = 0;
    uint8_t *stage_x = nullptr;     // device staging for the host-buffer entry point
    uint8_t *stage_y = nullptr;
    size_t stage_x_bytes = 0, stage_y_bytes = 0;
    uint8_t *bw_scratch = nullptr;  // transposed factors for the input gradient
    size_t bw_scratch_bytes = 0;
    int forced_path = 0;            // 0 auto, 1 simt, 2 decode (reassociated form), 3 umma (scale-MMA form), 4 decode16
    int forced_splitk = 0;          // 0 auto
    int forced_bn = 0;              // 0 auto; else the token tile of the scale-MMA kernel (32, 64, 128, 256)
    int last_cuda_error = 0;
    int last_launches = 0;
    const char *last_path = "none";
};

State &state();

// Records a failed CUDA call and maps it to LORDS_ERR_CUDA.
int cuda_fail(cudaError_t e);

#define LORDS_CUDA_TRY(expr)                                   \
    do {                                                       \
        cudaError_t e__ = (expr);                              \
        if (e__ != cudaSuccess) return ::lords::cuda_fail(e__);\
    } while (0)

// Generic CUDA-core path: any shape the interface accepts.
int launch_simt(const Problem &p, State &st, cudaStream_t stream);

// Tensor-core path (TMA + tcgen05/TMEM), scale matrix rebuilt per tile by a small MMA.
// LORDS_ERR_UNSUPPORTED for shapes outside its rules.
int launch_umma(const Problem &p, State &st, cudaStream_t stream);

// Tensor-core decode path (M <= 2), reassociated form with the scale factors folded into the
// activation operand.  LORDS_ERR_UNSUPPORTED for shapes outside its rules.
int launch_decode(const Problem &p, State &st, cudaStream_t stream);

// Tensor-core decode path for 3 .. 16 tokens, scale-MMA form with 128-column k-steps.
// LORDS_ERR_UNSUPPORTED for shapes outside its rules.
int launch_decode16(const Problem &p, State &st, cudaStream_t stream);

// Quantisation step (codes from W, B, A): tensor-core kernel where its rules hold, CUDA cores otherwise.
int launch_quantize(const void *W, const void *B, const void *A, const float *levels, int bits, int m, int n, int r,
                    uint8_t *Q, State &st, cudaStream_t stream);

// Backward with the codes fixed (Sec. 3.4): transposition of packed codes and of a bf16 matrix (what the
// input gradient needs to run on the forward kernels), and the gradients of B and A on the CUDA cores.
int launch_transpose_codes(const uint8_t *Q, int m, int n, int bits, uint8_t *Qt, cudaStream_t stream);
int launch_transpose_bf16_pair(const uint16_t *src0, int rows0, int cols0, uint16_t *dst0, const uint16_t *src1, int rows1, int cols1,
                               uint16_t *dst1, cudaStream_t stream);
int launch_backward_factors(const uint16_t *g, const uint16_t *x, const uint8_t *q, const uint16_t *B, const uint16_t *A,
                            const float *levels, int bits, int M, int m, int n, int r, float *dB, float *dA,
                            State &st, cudaStream_t stream);

// Straight-through gradients of quantisation-aware training (Eq. 4-5): the tensor-core schedule where its
// rules hold, else one pass over W per requested factor gradient on the CUDA cores.
int launch_backward_qat(const uint16_t *g, const uint16_t *x, const uint16_t *W, const uint8_t *q, const uint16_t *B,
                        const uint16_t *A, const float *levels, int bits, int M, int m, int n, int r, float *dW, float *dB,
                        float *dA, State &st, cudaStream_t stream);

// Comparators (Sec. 4.4, Table 6): the block-scale instantiation of the 16-token decode kernel (Eq. 2) and
// the two extra launches of an additive low-rank adapter on top of it.
int launch_blockscale16(const Problem &p, const uint16_t *scales, int blk, State &st, cudaStream_t stream);
int launch_adapter(const uint16_t *x, const uint16_t *Al, const uint16_t *Bl, const float *y32, float *u, void *y, int y_f32,
                   int M, int m, int n, int r, cudaStream_t stream);

}  // namespace lords
