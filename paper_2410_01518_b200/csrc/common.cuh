// Shared device helpers of the memory-pot kernels.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ipotk {

// Sticky device status values (mirrors of IPOT_E_TIMEOUT / IPOT_E_BOUNDS).
constexpr int kStatusTimeout = -5;
constexpr int kStatusBounds = -6;

__device__ __forceinline__ void set_status(int *status, int code)
{
    if (status) atomicCAS(status, 0, code);
}

// Monotone map float -> uint32: a < b  <=>  key(a) < key(b) (for non-NaN values).
__device__ __forceinline__ uint32_t order_key(float f)
{
    uint32_t b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// One 16-byte vector of storage elements -> floats.
template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int kElems = 4;
    __device__ static __forceinline__ void load(const float *p, float *out)
    {
        float4 v = *reinterpret_cast<const float4 *>(p);
        out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int kElems = 8;
    __device__ static __forceinline__ void load(const __nv_bfloat16 *p, float *out)
    {
        uint4 v = *reinterpret_cast<const uint4 *>(p);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            out[2 * i] = __uint_as_float(w[i] << 16);
            out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
};

}  // namespace ipotk
