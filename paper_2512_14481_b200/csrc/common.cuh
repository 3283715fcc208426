// Shared host/device helpers of the SASQ sm_100a library (no method arithmetic
// beyond the 16-bit storage conversions).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstddef>
#include <cstdint>

#include "../../include/sasq.h"

namespace sasq {

// ---------------------------------------------------------------------------
// device status word: one per translation unit that needs it, read and cleared
// by sasq_device_status through the readers below.
// ---------------------------------------------------------------------------
#define SASQ_DEFINE_STATUS_WORD(name)                                                        \
    static __device__ int name = 0;                                                          \
    static inline int name##_read_and_clear(cudaStream_t st) {                               \
        int h = 0, z = 0;                                                                    \
        if (cudaMemcpyFromSymbolAsync(&h, name, sizeof(int), 0, cudaMemcpyDeviceToHost, st)  \
            != cudaSuccess) return SASQ_ERR_CUDA;                                            \
        if (cudaStreamSynchronize(st) != cudaSuccess) return SASQ_ERR_CUDA;                  \
        if (h != 0) {                                                                        \
            if (cudaMemcpyToSymbolAsync(name, &z, sizeof(int), 0, cudaMemcpyHostToDevice, st)\
                != cudaSuccess) return SASQ_ERR_CUDA;                                        \
            if (cudaStreamSynchronize(st) != cudaSuccess) return SASQ_ERR_CUDA;              \
        }                                                                                    \
        return h;                                                                            \
    }

// ---------------------------------------------------------------------------
// Programmatic dependent launch.  The hot kernels are launched with the
// programmatic-stream-serialization attribute: the next kernel of the stream may
// be scheduled while this one still runs (as SMs free up) and does its set-up,
// then waits here until every kernel before it has completed and its memory is
// visible.  Nothing that an earlier kernel may have written (or may still read)
// is touched before pdl_wait().  Without the attribute both are no-ops.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void pdl_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ bool scale_is_bad(float s) {
    const float inv = __fdiv_rn(1.0f, s);
    return !(s == s) || s == 0.0f || isinf(s) || isinf(inv) || !(inv == inv);
}

// ---------------------------------------------------------------------------
// 16-bit storage: two values per 32-bit word, low half first.
// ---------------------------------------------------------------------------
template <bool BF>
__device__ __forceinline__ float2 widen2(uint32_t w) {
    if constexpr (BF) {
        return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
    } else {
        return __half22float2(*reinterpret_cast<const __half2*>(&w));
    }
}

template <bool BF>
__device__ __forceinline__ float widen1(uint16_t h) {
    if constexpr (BF) {
        return __uint_as_float((uint32_t)h << 16);
    } else {
        return __half2float(__ushort_as_half(h));
    }
}

// one round-to-nearest-even narrowing per value
template <bool BF>
__device__ __forceinline__ uint32_t narrow2(float lo, float hi) {
    if constexpr (BF) {
        __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&v);
    } else {
        __half2 v = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&v);
    }
}

template <bool BF>
__device__ __forceinline__ uint16_t narrow1(float f) {
    if constexpr (BF) {
        return __bfloat16_as_ushort(__float2bfloat16_rn(f));
    } else {
        return __half_as_ushort(__float2half_rn(f));
    }
}

// ---------------------------------------------------------------------------
// host-side checks
// ---------------------------------------------------------------------------
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// launch attribute that lets a kernel start its set-up under the tail of the kernel before it in the stream
inline cudaLaunchAttribute pdl_attribute() {
    cudaLaunchAttribute a{};
    a.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    a.val.programmaticStreamSerializationAllowed = 1;
    return a;
}

// SM count of the current device if it is sm_100 (compute capability 10.x), else <= 0.
int device_sm_count_if_sm100();

}  // namespace sasq
