// Token novelty (Sec. 3.3.2, Eq. 3): n_t = -log softmax(z_t)[x_t] for the model's logits z_t over the
// vocabulary and the token x_t that actually followed - the per-token cross-entropy whose largest values
// the NuC criterion keeps.  One pass over the logits, HBM-bound: V * e bytes per token.
//
// novelty_kernel, grid (segments, tokens): a block of 128 threads reads one segment of 8192 logits of one row
// with 16-byte loads (eight per thread in flight) and reduces it to (reference, sum 2^(z log2e - reference)), the reference being the segment's largest
// logit in log2 units.  Rows are cut into segments so that the grid is fine-grained (a whole 32k-256k row per
// block would leave a long tail on 148 SMs).  The block that finishes a row last (a counter per row, no
// waiting) merges the row's segments, fetches the label's logit and writes log-sum-exp minus it to the
// token's slot of the novelty array.
//
// One exponential per logit is the floor of the arithmetic (16 per clock per SM: 0.7 of the time the HBM
// transfer takes for bf16), so everything around it is packed: the maximum of a 16-byte group is taken on the
// bf16 pairs, once per batch of loads, the scale-and-shift is one packed FMA per pair, the sums are packed
// adds, and the block reduction spends one exponential per thread.
#pragma once
#include <cuda_bf16.h>

#include "common.cuh"

namespace ipotk {

constexpr int kNovThreads = 128;
constexpr int kNovBatch = 8;          // 16-byte loads a thread has in flight
constexpr int kNovSegElems = 8192;
constexpr int kNovMaxRows = 65535;   // tokens per call (grid y limit); the row counters are sized for it
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float nov_ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float nov_max3(float a, float b, float c)
{
    float y;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
    return y;
}

// Running statistics of a thread: ref = fl(largest logit seen * log2e), the exponent every term is taken
// relative to, s = sum of 2^(z log2e - ref) in two lanes for the packed adds.
struct NovStat {
    float ref;
    float2 s;
    // lm = largest logit of the values added next; no branch: the factor is 1 when the reference stays
    __device__ __forceinline__ void raise(float lm)
    {
        const float nref = fmaxf(ref, lm * kLog2e);
        const float f = nov_ex2(ref - nref);  // first time: ref = -inf, f = 0, s is 0 anyway
        s = __fmul2_rn(s, make_float2(f, f));
        ref = nref;
    }
    __device__ __forceinline__ void add_pair(float2 z)
    {
        const float2 t = __ffma2_rn(z, make_float2(kLog2e, kLog2e), make_float2(-ref, -ref));
        s = __fadd2_rn(s, make_float2(nov_ex2(t.x), nov_ex2(t.y)));
    }
    __device__ __forceinline__ void add_one(float z)
    {
        raise(z);
        s.x += nov_ex2(fmaf(z, kLog2e, -ref));
    }
};

// (ref, sum) pairs relative to their own reference -> relative to the larger one
__device__ __forceinline__ void nov_merge(float &ref, float &sum, float ref2, float sum2)
{
    const float rn = fmaxf(ref, ref2);
    const float a = (ref == -INFINITY) ? 0.f : sum * nov_ex2(ref - rn);
    const float b = (ref2 == -INFINITY) ? 0.f : sum2 * nov_ex2(ref2 - rn);
    ref = rn;
    sum = a + b;
}

__device__ __forceinline__ float nov_load1(const float *p) { return __ldg(p); }
__device__ __forceinline__ float nov_load1(const __nv_bfloat16 *p) { return __bfloat162float(*p); }

// largest logit of kNovBatch 16-byte groups
__device__ __forceinline__ float nov_batch_max(const uint4 (&v)[kNovBatch], const float *)
{
    float m = -INFINITY;
#pragma unroll
    for (int u = 0; u < kNovBatch; ++u) {
        m = nov_max3(m, __uint_as_float(v[u].x), __uint_as_float(v[u].y));
        m = nov_max3(m, __uint_as_float(v[u].z), __uint_as_float(v[u].w));
    }
    return m;
}
__device__ __forceinline__ float nov_batch_max(const uint4 (&v)[kNovBatch], const __nv_bfloat16 *)
{
    // on the bf16 pairs: exact, and half the instructions
    auto h2 = [](const uint32_t &w) { return *reinterpret_cast<const __nv_bfloat162 *>(&w); };
    __nv_bfloat162 m = __hmax2(__hmax2(h2(v[0].x), h2(v[0].y)), __hmax2(h2(v[0].z), h2(v[0].w)));
#pragma unroll
    for (int u = 1; u < kNovBatch; ++u) m = __hmax2(__hmax2(m, h2(v[u].x)), __hmax2(__hmax2(h2(v[u].y), h2(v[u].z)), h2(v[u].w)));
    return fmaxf(__low2float(m), __high2float(m));
}
// the terms of one 16-byte group into one of the thread's accumulators
__device__ __forceinline__ void nov_group(NovStat &st, const uint4 &v, const float *)
{
    st.add_pair(make_float2(__uint_as_float(v.x), __uint_as_float(v.y)));
    st.add_pair(make_float2(__uint_as_float(v.z), __uint_as_float(v.w)));
}
__device__ __forceinline__ void nov_group(NovStat &st, const uint4 &v, const __nv_bfloat16 *)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) st.add_pair(make_float2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xffff0000u)));
}

// grid (segs, rows), block 128.  counters: [rows] ints, zero on entry and zero again on exit; partial: [rows][segs].
// Token `row` = (stream b, position t) = (row / n_tokens, row % n_tokens) writes out[b * out_stride + slot0 + t].
// A negative label marks an ignored position (novelty 0); a label >= V also gives 0 and raises kStatusBounds.
template <typename T>
__global__ void __launch_bounds__(kNovThreads)
novelty_kernel(const T *__restrict__ logits, size_t row_stride, int V, int segs, float2 *partial, int *counters,
               const int32_t *__restrict__ labels, int n_tokens, float *__restrict__ out, size_t out_stride, int slot0,
               int *status)
{
    constexpr int VE = 16 / (int)sizeof(T);
    const int seg = blockIdx.x;
    const size_t row = blockIdx.y;
    const int v0 = seg * kNovSegElems, v1 = min(V, v0 + kNovSegElems);
    const T *z = logits + row * row_stride;
    NovStat st{-INFINITY, make_float2(0.f, 0.f)};
    if ((reinterpret_cast<uintptr_t>(z) & 15u) == 0) {
        // 16-byte loads, kNovBatch per thread in flight; one reference update per batch
        const int nvec = (v1 - v0) / VE;
        const uint4 *zv = reinterpret_cast<const uint4 *>(z + v0);
        constexpr uint32_t kNegInf = sizeof(T) == 2 ? 0xFF80FF80u : 0xFF800000u;  // -inf: no term, never the maximum
        for (int i0 = 0; i0 + (int)threadIdx.x < nvec; i0 += kNovBatch * kNovThreads) {  // this thread has >= 1 group
            uint4 v[kNovBatch];
#pragma unroll
            for (int u = 0; u < kNovBatch; ++u) {
                const int i = i0 + u * kNovThreads + threadIdx.x;
                v[u] = i < nvec ? __ldcs(zv + i) : make_uint4(kNegInf, kNegInf, kNegInf, kNegInf);  // streamed once
            }
            st.raise(nov_batch_max(v, z));
#pragma unroll
            for (int u = 0; u < kNovBatch; ++u) nov_group(st, v[u], z);
        }
        for (int i = v0 + nvec * VE + threadIdx.x; i < v1; i += kNovThreads) st.add_one(nov_load1(z + i));  // < VE elements
    } else {  // a row that does not start on a 16-byte boundary: element loads
        for (int i = v0 + threadIdx.x; i < v1; i += kNovThreads) st.add_one(nov_load1(z + i));
    }
    // block reduction in two steps (largest reference, then the sums rescaled once): one exponential per thread
    __shared__ float wred[2][kNovThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float ref = st.ref;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) ref = fmaxf(ref, __shfl_xor_sync(0xffffffffu, ref, off));
    if (lane == 0) wred[0][warp] = ref;
    __syncthreads();
    ref = wred[0][0];
#pragma unroll
    for (int w = 1; w < kNovThreads / 32; ++w) ref = fmaxf(ref, wred[0][w]);
    float sum = (st.ref == -INFINITY) ? 0.f : (st.s.x + st.s.y) * nov_ex2(st.ref - ref);
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    if (lane == 0) wred[1][warp] = sum;
    __syncthreads();
    if (threadIdx.x != 0) return;
    sum = wred[1][0];
#pragma unroll
    for (int w = 1; w < kNovThreads / 32; ++w) sum += wred[1][w];
    if (segs > 1) {
        __stcg(&partial[row * segs + seg], make_float2(ref, sum));
        __threadfence();
        if (atomicAdd(&counters[row], 1) != segs - 1) return;  // another block finishes the row
        __threadfence();
        counters[row] = 0;  // ready for the next call
        ref = -INFINITY;
        sum = 0.f;
        for (int s = 0; s < segs; ++s) {
            const float2 p = __ldcg(&partial[row * segs + s]);
            nov_merge(ref, sum, p.x, p.y);
        }
    }
    const int label = labels[row];
    float nov = 0.f;
    if (label >= 0 && label < V)
        nov = kLn2 * ((ref - nov_load1(z + label) * kLog2e) + log2f(sum));  // log-sum-exp minus the label's logit
    else if (label >= V)
        set_status(status, kStatusBounds);
    out[(row / n_tokens) * out_stride + slot0 + row % n_tokens] = nov;
}

}  // namespace ipotk
