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

// ------------------------------------------------------------------ 2^t on the FMA pipe
// The scorers' softmax costs one exponential per logit and the special-function unit delivers 16 a clock per SM;
// a share of them is evaluated with ordinary arithmetic instead (Cody-Waite split at the rounding constant
// 1.5 * 2^23, degree-4 polynomial for 2^f on [-0.5, 0.5], relative error 2.7e-6, exponent added as an integer).
// 2^t for a pair, t <= 8, on the FMA pipe.  t is clamped at -126: with j = round(t) >= -126 and the polynomial in
// [0.707, 1.415] the exponent field of the result stays >= 0.  Results below 2^-126 (the clamp included: the
// polynomial is just below 1 at f = 0) come out as subnormal bit patterns; callers add them with flush-to-zero
// arithmetic or against sums that hold a far larger term, which matches the special-function unit's zero.
__device__ __forceinline__ float2 exp2_fma_pair(float2 t)
{
    t.x = fmaxf(t.x, -126.f);
    t.y = fmaxf(t.y, -126.f);
    const float2 magic = make_float2(12582912.f, 12582912.f);       // 1.5 * 2^23: adding it rounds t to an integer
    const float2 r = __fadd2_rn(t, magic);
    const float2 jf = __fadd2_rn(r, make_float2(-12582912.f, -12582912.f));
    const float2 f = __ffma2_rn(jf, make_float2(-1.f, -1.f), t);    // in [-0.5, 0.5]
    float2 p = __ffma2_rn(make_float2(0.009570101276f, 0.009570101276f), f, make_float2(0.05591785908f, 0.05591785908f));
    p = __ffma2_rn(p, f, make_float2(0.2402474433f, 0.2402474433f));
    p = __ffma2_rn(p, f, make_float2(0.6931217909f, 0.6931217909f));
    p = __ffma2_rn(p, f, make_float2(0.9999992847f, 0.9999992847f));
    // the integer sits in the low mantissa bits of r; the shift drops the rest of r
    return make_float2(__int_as_float(__float_as_int(p.x) + (__float_as_int(r.x) << 23)),
                       __int_as_float(__float_as_int(p.y) + (__float_as_int(r.y) << 23)));
}
// Pair i of a piece goes to the FMA pipe if its position in an evenly spread order of 8 is below kPoly.
template <int kPoly>
__device__ __forceinline__ constexpr bool pair_on_fma(int i)
{
    constexpr int order[8] = {0, 4, 2, 6, 1, 5, 3, 7};
    return order[i & 7] < kPoly;
}

}  // namespace ipotk
