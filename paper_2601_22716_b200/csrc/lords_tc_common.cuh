// Host-side helpers shared by the tensor-core translation units: the tensor-map encoder with a
// small cache, the output store, and per-device bookkeeping for launch attributes.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <mutex>

#include "lords_internal.h"

namespace lords {

constexpr int kMaxDevices = 64;   // per-device caches are indexed by the CUDA device ordinal

// Index of the library's device in the per-device caches (0 when out of range: such a device
// simply shares slot 0 and re-applies its attributes).
inline int device_slot(const State &st) { return st.device >= 0 && st.device < kMaxDevices ? st.device : 0; }

__device__ __forceinline__ void store_out(void *y, int y_f32, size_t idx, float v)
{
    if (y_f32) static_cast<float *>(y)[idx] = v;
    else static_cast<__nv_bfloat16 *>(y)[idx] = __float2bfloat16_rn(v);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn()
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

// A 2-D tiled tensor map over a dense row-major matrix (`inner` elements per row, `outer` rows),
// box {box_inner, box_outer}, out-of-bounds elements read as zero.  A tensor map is a pure function
// of these arguments, so the encoded maps of the layers seen so far are kept in a direct-mapped
// cache: a layer that is called again encodes nothing.
inline bool make_map_2d(CUtensorMap *map, CUtensorMapDataType dt, int elem_bytes, const void *ptr, uint64_t inner,
                        uint64_t outer, uint32_t box_inner, uint32_t box_outer, CUtensorMapSwizzle swz)
{
    struct Key {
        const void *ptr;
        uint64_t inner, outer;
        uint32_t box_inner, box_outer;
        int dt, swz;
    };
    struct Entry {
        Key key;
        bool valid;
        CUtensorMap map;
    };
    constexpr int kSlots = 4096;
    static Entry *cache = new Entry[kSlots]();
    static std::mutex mu;
    Key key;
    memset(&key, 0, sizeof(key));
    key.ptr = ptr; key.inner = inner; key.outer = outer; key.box_inner = box_inner; key.box_outer = box_outer;
    key.dt = (int)dt; key.swz = (int)swz;
    uint64_t h = reinterpret_cast<uintptr_t>(ptr) * 0x9E3779B97F4A7C15ull;
    h ^= (inner * 0xC2B2AE3D27D4EB4Full) ^ (outer * 0x165667B19E3779F9ull) ^ ((uint64_t)box_inner << 40) ^
         ((uint64_t)box_outer << 20) ^ ((uint64_t)swz << 8) ^ (uint64_t)dt;
    Entry &e = cache[(h >> 32) % kSlots];
    std::lock_guard<std::mutex> lock(mu);
    if (e.valid && memcmp(&e.key, &key, sizeof(Key)) == 0) {
        *map = e.map;
        return true;
    }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {inner * (uint64_t)elem_bytes};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    if (fn(map, dt, 2, const_cast<void *>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
           CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    e.key = key;
    e.map = *map;
    e.valid = true;
    return true;
}

}  // namespace lords
