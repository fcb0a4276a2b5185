// Generation over the pot: one new query per query head attends to the rows of its KV head's unit (after CCD
// the heads of a layer keep different tokens, Sec. 3.3.1, so every unit is its own little cache; Sec. 4.5
// measures generation at a fixed pot).  out_h = sum_j softmax_j(q_h . k_j / sqrt(d)) v_j, plus the log-sum-exp
// so that a caller can merge the result with attention over tokens that are not in the pot.
//
// With G = Hq / Hkv <= 8 query rows per unit this is a pure HBM stream (every K and V row is read once:
// 2 * len * d * e bytes per unit), so no tensor cores: a group of `lpk` lanes (one 16-byte vector of the row each)
// owns a key, dots its slice with the G queries kept in registers, and the slice sums are added across the
// group with shuffles.  Keys are taken in tiles of KT per group: KT key loads in flight, one rescale of the
// running output per tile, then KT value loads.  grid (splits, units): a block covers a range of the unit's rows;
// the block that finishes a unit last (a counter per unit, no waiting) merges the splits.
#pragma once
#include "common.cuh"
#include "k_rope.cuh"  // RopeVec: 16-byte vector <-> floats

namespace ipotk {

constexpr int kDecThreads = 256;
constexpr int kDecWarps = kDecThreads / 32;

__device__ __forceinline__ float dec_ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// 2^(m - ref) with "nothing seen yet" (m = -inf) giving 0 whatever ref is
__device__ __forceinline__ float dec_scale(float m, float ref) { return m == -INFINITY ? 0.f : dec_ex2(m - ref); }

__host__ __device__ inline size_t decode_smem_bytes(int G, int d) { return (size_t)kDecWarps * G * (d + 2) * sizeof(float); }

// partial: [units][splits][G][d + 2] floats (unnormalised output, then reference exponent and sum, log2 units);
// counters: [units] ints, zero on entry and zero again on exit.  lpk = 16-byte vectors per row (4, 8, 16 or 32).
template <typename T, int G, int KT>
__global__ void __launch_bounds__(kDecThreads)
decode_attn_kernel(const T *__restrict__ Kp, const T *__restrict__ Vp, const T *__restrict__ q, float *__restrict__ out,
                   float *__restrict__ lse, float *partial, int *counters, int N, int d, int lpk, size_t unit_elems, float scale_log2e)
{
    constexpr int VE = RopeVec<T>::kElems;
    extern __shared__ __align__(16) float dec_sm[];  // [warps][G][d + 2]
    __shared__ int is_last;
    const int unit = blockIdx.y, split = blockIdx.x, splits = gridDim.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gq = lane / lpk, gl = lane - gq * lpk, gpw = 32 / lpk, ng = kDecWarps * gpw, grp = warp * gpw + gq;
    const int per = (N + splits - 1) / splits, k0 = split * per, k1 = min(N, k0 + per);
    const T *Ku = Kp + (size_t)unit * unit_elems + gl * VE, *Vu = Vp + (size_t)unit * unit_elems + gl * VE;

    float qf[G][VE], acc[G][VE], m[G], l[G];
#pragma unroll
    for (int h = 0; h < G; ++h) {
        RopeVec<T>::unpack(__ldg(reinterpret_cast<const uint4 *>(q + ((size_t)unit * G + h) * d + gl * VE)), qf[h]);
#pragma unroll
        for (int i = 0; i < VE; ++i) {
            qf[h][i] *= scale_log2e;
            acc[h][i] = 0.f;
        }
        m[h] = -INFINITY;
        l[h] = 0.f;
    }

    for (int base = k0; base < k1; base += ng * KT) {  // the same trip count for every lane of the block
        uint4 kv[KT];
        bool valid[KT];
#pragma unroll
        for (int j = 0; j < KT; ++j) {
            const int key = base + j * ng + grp;
            valid[j] = key < k1;
            kv[j] = valid[j] ? __ldcs(reinterpret_cast<const uint4 *>(Ku + (size_t)key * d)) : make_uint4(0, 0, 0, 0);
        }
        float s[KT][G];
#pragma unroll
        for (int j = 0; j < KT; ++j) {
            float x[VE];
            RopeVec<T>::unpack(kv[j], x);
#pragma unroll
            for (int h = 0; h < G; ++h) {
                float a = 0.f;
#pragma unroll
                for (int i = 0; i < VE; ++i) a = fmaf(x[i], qf[h][i], a);
                s[j][h] = a;
            }
        }
        // the value rows are requested before the scores are finished
        uint4 vv[KT];
#pragma unroll
        for (int j = 0; j < KT; ++j) {
            const int key = base + j * ng + grp;
            vv[j] = valid[j] ? __ldcs(reinterpret_cast<const uint4 *>(Vu + (size_t)key * d)) : make_uint4(0, 0, 0, 0);
        }
        for (int off = lpk >> 1; off >= 1; off >>= 1) {
#pragma unroll
            for (int j = 0; j < KT; ++j)
#pragma unroll
                for (int h = 0; h < G; ++h) s[j][h] += __shfl_xor_sync(0xffffffffu, s[j][h], off);
        }
        float corr[G];
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float mt = -INFINITY;
#pragma unroll
            for (int j = 0; j < KT; ++j) mt = fmaxf(mt, valid[j] ? s[j][h] : -INFINITY);
            const float mn = fmaxf(m[h], mt);
            corr[h] = dec_scale(m[h], mn);
            m[h] = mn;
            float ls = 0.f;
#pragma unroll
            for (int j = 0; j < KT; ++j) {
                s[j][h] = valid[j] ? dec_ex2(s[j][h] - mn) : 0.f;  // now the weight of key j
                ls += s[j][h];
            }
            l[h] = fmaf(l[h], corr[h], ls);
#pragma unroll
            for (int i = 0; i < VE; ++i) acc[h][i] *= corr[h];
        }
#pragma unroll
        for (int j = 0; j < KT; ++j) {
            float x[VE];
            RopeVec<T>::unpack(vv[j], x);
#pragma unroll
            for (int h = 0; h < G; ++h)
#pragma unroll
                for (int i = 0; i < VE; ++i) acc[h][i] = fmaf(s[j][h], x[i], acc[h][i]);
        }
    }

    // ---- the groups of a warp (they hold different keys, the same channels)
    for (int off = lpk; off < 32; off <<= 1) {
#pragma unroll
        for (int h = 0; h < G; ++h) {
            const float m2 = __shfl_xor_sync(0xffffffffu, m[h], off), l2 = __shfl_xor_sync(0xffffffffu, l[h], off);
            const float mn = fmaxf(m[h], m2);
            const float ca = dec_scale(m[h], mn), cb = dec_scale(m2, mn);
            l[h] = l[h] * ca + l2 * cb;
            m[h] = mn;
#pragma unroll
            for (int i = 0; i < VE; ++i) acc[h][i] = acc[h][i] * ca + __shfl_xor_sync(0xffffffffu, acc[h][i], off) * cb;
        }
    }
    // ---- the warps of the block, through shared memory
    const int ds = d + 2;
    if (gq == 0) {
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float *row = dec_sm + ((size_t)warp * G + h) * ds;
#pragma unroll
            for (int i = 0; i < VE; ++i) row[gl * VE + i] = acc[h][i];
            if (gl == 0) {
                row[d] = m[h];
                row[d + 1] = l[h];
            }
        }
    }
    __syncthreads();
    float *dst = partial + ((size_t)unit * splits + split) * G * ds;
    for (int e = threadIdx.x; e < G * ds; e += kDecThreads) {
        const int h = e / ds, c = e - h * ds;
        float ref = -INFINITY;
#pragma unroll
        for (int w = 0; w < kDecWarps; ++w) ref = fmaxf(ref, dec_sm[((size_t)w * G + h) * ds + d]);
        float v;
        if (c == d) {
            v = ref;
        } else {
            v = 0.f;
#pragma unroll
            for (int w = 0; w < kDecWarps; ++w) {
                const float *row = dec_sm + ((size_t)w * G + h) * ds;
                v = fmaf(row[c], dec_scale(row[d], ref), v);
            }
        }
        __stcg(dst + e, v);
    }
    // ---- the splits of the unit: the block that arrives last merges them
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const int done = splits > 1 ? atomicAdd(&counters[unit], 1) : 0;
        is_last = done == splits - 1;
        if (is_last && splits > 1) counters[unit] = 0;  // ready for the next call
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const float *src = partial + (size_t)unit * splits * G * ds;
    for (int e = threadIdx.x; e < G * d; e += kDecThreads) {
        const int h = e / d, c = e - h * d;
        float ref = -INFINITY;
        for (int sp = 0; sp < splits; ++sp) ref = fmaxf(ref, __ldcg(src + ((size_t)sp * G + h) * ds + d));
        float o = 0.f, den = 0.f;
        for (int sp = 0; sp < splits; ++sp) {
            const float *row = src + ((size_t)sp * G + h) * ds;
            const float w = dec_scale(__ldcg(row + d), ref);
            o = fmaf(__ldcg(row + c), w, o);
            den = fmaf(__ldcg(row + d + 1), w, den);
        }
        out[((size_t)unit * G + h) * d + c] = o / den;
        if (c == 0 && lse) lse[(size_t)unit * G + h] = 0.6931471805599453f * (ref + log2f(den));
    }
}

}  // namespace ipotk
