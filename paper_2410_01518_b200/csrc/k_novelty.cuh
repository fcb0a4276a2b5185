// Token novelty (Sec. 3.3.2, Eq. 3): n_t = -log softmax(z_t)[x_t] for the model's logits z_t over the
// vocabulary and the token x_t that actually followed - the per-token cross-entropy whose largest values
// the NuC criterion keeps.  One pass over the logits, HBM-bound: V * e bytes per token.
//   novelty_partial_kernel : grid (segments, tokens); a block reads one segment of 8192 logits of one row
//                            with 16-byte loads and reduces it to (max, sum 2^(x - max)) in log2 units.
//                            Rows are cut into segments so that the grid is fine-grained (a whole 32k-256k
//                            row per block would leave a long tail on 148 SMs).
//   novelty_finish_kernel  : one thread per token merges the row's segments, fetches the label's logit
//                            and writes log-sum-exp minus it to the token's slot of the novelty array.
#pragma once
#include <cuda_bf16.h>

#include "common.cuh"

namespace ipotk {

constexpr int kNovThreads = 256;
constexpr int kNovSegElems = 8192;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float nov_ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Running (max, sum 2^(x - max)) of a thread; all values in log2 units.
struct NovStat {
    float m, s;
    __device__ __forceinline__ void add_group(const float *x, int n)
    {
        float lm = x[0];
        for (int i = 1; i < n; ++i) lm = fmaxf(lm, x[i]);
        if (lm > m) {
            s *= nov_ex2(m - lm);  // m = -inf: s is 0 and stays 0
            m = lm;
        }
        for (int i = 0; i < n; ++i) s += nov_ex2(x[i] - m);
    }
    __device__ __forceinline__ void merge(float m2, float s2)
    {
        const float mn = fmaxf(m, m2);
        const float a = (m == -INFINITY) ? 0.f : s * nov_ex2(m - mn);
        const float b = (m2 == -INFINITY) ? 0.f : s2 * nov_ex2(m2 - mn);
        m = mn;
        s = a + b;
    }
};

__device__ __forceinline__ float nov_load1(const float *p) { return __ldg(p) * kLog2e; }
__device__ __forceinline__ float nov_load1(const __nv_bfloat16 *p) { return __bfloat162float(*p) * kLog2e; }

template <typename T> struct NovVec;
template <> struct NovVec<float> {
    static constexpr int kElems = 4;
    __device__ static void unpack(const uint4 &v, float *x)
    {
        x[0] = __uint_as_float(v.x) * kLog2e; x[1] = __uint_as_float(v.y) * kLog2e;
        x[2] = __uint_as_float(v.z) * kLog2e; x[3] = __uint_as_float(v.w) * kLog2e;
    }
};
template <> struct NovVec<__nv_bfloat16> {
    static constexpr int kElems = 8;
    __device__ static void unpack(const uint4 &v, float *x)
    {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16) * kLog2e;
            x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u) * kLog2e;
        }
    }
};

// grid (segs, rows).  partial[row * segs + seg] = (max, sum) of logits[row][seg * 8192 ...) in log2 units.
template <typename T>
__global__ void __launch_bounds__(kNovThreads)
novelty_partial_kernel(const T *__restrict__ logits, size_t row_stride, int V, int segs, float2 *__restrict__ partial)
{
    constexpr int VE = NovVec<T>::kElems;
    const int seg = blockIdx.x;
    const size_t row = blockIdx.y;
    const int v0 = seg * kNovSegElems, v1 = min(V, v0 + kNovSegElems);
    const T *z = logits + row * row_stride;
    NovStat st{-INFINITY, 0.f};
    if ((reinterpret_cast<uintptr_t>(z) & 15u) == 0) {
        // 16-byte loads; four per thread are issued before any is used
        const int nvec = (v1 - v0) / VE;
        const uint4 *zv = reinterpret_cast<const uint4 *>(z + v0);
        for (int i0 = 0; i0 < nvec; i0 += 4 * kNovThreads) {
            uint4 v[4];
            bool have[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u * kNovThreads + threadIdx.x;
                have[u] = i < nvec;
                if (have[u]) v[u] = __ldcs(zv + i);  // streamed once: evict first
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (have[u]) {
                    float x[VE];
                    NovVec<T>::unpack(v[u], x);
                    st.add_group(x, VE);
                }
            }
        }
        for (int i = v0 + nvec * VE + threadIdx.x; i < v1; i += kNovThreads) {  // fewer than VE elements
            const float x = nov_load1(z + i);
            st.add_group(&x, 1);
        }
    } else {  // a row that does not start on a 16-byte boundary: element loads
        for (int i = v0 + threadIdx.x; i < v1; i += kNovThreads) {
            const float x = nov_load1(z + i);
            st.add_group(&x, 1);
        }
    }
    // block reduction
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, st.m, off);
        const float s2 = __shfl_xor_sync(0xffffffffu, st.s, off);
        st.merge(m2, s2);
    }
    __shared__ float2 wst[kNovThreads / 32];
    if ((threadIdx.x & 31) == 0) wst[threadIdx.x >> 5] = make_float2(st.m, st.s);
    __syncthreads();
    if (threadIdx.x == 0) {
        NovStat t{wst[0].x, wst[0].y};
#pragma unroll
        for (int w = 1; w < kNovThreads / 32; ++w) t.merge(wst[w].x, wst[w].y);
        partial[row * segs + seg] = make_float2(t.m, t.s);
    }
}

// grid (ceil(rows / 256)).  Token `row` = (stream b, position t) = (row / n_tokens, row % n_tokens) writes
// out[b * out_stride + slot0 + t].  A negative label marks an ignored position (novelty 0); a label >= V
// also gives 0 and raises kStatusBounds.
template <typename T>
__global__ void __launch_bounds__(kNovThreads)
novelty_finish_kernel(const T *__restrict__ logits, size_t row_stride, int V, int segs, const float2 *__restrict__ partial,
                      const int32_t *__restrict__ labels, size_t rows, int n_tokens, float *__restrict__ out,
                      size_t out_stride, int slot0, int *status)
{
    const size_t row = (size_t)blockIdx.x * kNovThreads + threadIdx.x;
    if (row >= rows) return;
    const int label = labels[row];
    float nov = 0.f;
    if (label >= 0 && label < V) {
        NovStat t{-INFINITY, 0.f};
        for (int s = 0; s < segs; ++s) {
            const float2 p = partial[row * segs + s];
            t.merge(p.x, p.y);
        }
        const float xl = nov_load1(logits + row * row_stride + label);
        nov = kLn2 * ((t.m - xl) + log2f(t.s));  // log-sum-exp minus the label's logit
    } else if (label >= V) {
        set_status(status, kStatusBounds);
    }
    out[(row / n_tokens) * out_stride + slot0 + row % n_tokens] = nov;
}

}  // namespace ipotk
