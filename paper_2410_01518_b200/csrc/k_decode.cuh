// Generation over the pot: one new query per query head attends to the rows of its KV head's unit (after CCD
// the heads of a layer keep different tokens, Sec. 3.3.1, so every unit is its own little cache; Sec. 4.5
// measures generation at a fixed pot).  out_h = sum_j softmax_j(q_h . k_j / sqrt(d)) v_j, plus the log-sum-exp
// so that a caller can merge the result with attention over tokens that are not in the pot.
//
// With G = Hq / Hkv <= 8 query rows per unit this is a pure HBM stream (every K and V row is read once:
// 2 * len * d * e bytes per unit), so no tensor cores.  grid (splits, units): a block covers a range of the
// unit's rows.  The rows arrive through a ring of shared-memory stages filled by cp.async (16 KiB of keys and
// 16 KiB of values per stage, two stages in flight while the third is used, two blocks per SM; a thread reads
// back exactly the vectors it copied, so the ring needs no barrier), so the stream does not wait for the arithmetic.  A group of `lpk` lanes (one 16-byte vector of the row each) owns a key: it dots its slice with
// the G queries kept in registers and the slice sums are added across the group with shuffles; a group takes
// four keys of a stage, rescales its running output only when a maximum moved, then adds the four value rows.
// The block that finishes a unit last (a counter per unit, no waiting) merges the splits.
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

constexpr int kDecKT = 4;                       // keys of a stage per lane group
constexpr int kDecStageVecs = kDecKT * kDecThreads;  // 16-byte vectors of keys (and of values) per stage: 16 KiB each
constexpr int kDecStages = 3;

__host__ __device__ inline size_t decode_smem_bytes(int G, int d)
{
    const size_t ring = (size_t)kDecStages * 2 * kDecStageVecs * 16, merge = (size_t)kDecWarps * G * (d + 2) * sizeof(float);
    return ring > merge ? ring : merge;
}

__device__ __forceinline__ void dec_cp_async16(void *smem_dst, const void *gmem_src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void dec_cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int kPending> __device__ __forceinline__ void dec_cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(kPending) : "memory"); }

// partial: [units][splits][G][d + 2] floats (unnormalised output, then reference exponent and sum, log2 units);
// counters: [units] ints, zero on entry and zero again on exit.  lpk = 16-byte vectors per row (4, 8, 16 or 32).
template <typename T, int G>
__global__ void __launch_bounds__(kDecThreads, G <= 4 ? 2 : 1)  // two blocks per SM: one streams while the other starts or merges
decode_attn_kernel(const T *__restrict__ Kp, const T *__restrict__ Vp, const T *__restrict__ q, float *__restrict__ out,
                   float *__restrict__ lse, float *partial, int *counters, int N, int d, int lpk, size_t unit_elems, float scale_log2e)
{
    constexpr int VE = RopeVec<T>::kElems;
    constexpr int KT = kDecKT;
    extern __shared__ __align__(16) uint8_t dec_raw[];
    uint4 *ring = reinterpret_cast<uint4 *>(dec_raw);   // [stages][K | V][kDecStageVecs]
    float *dec_sm = reinterpret_cast<float *>(dec_raw); // after the stream: [warps][G][d + 2]
    __shared__ int is_last;
    const int unit = blockIdx.y, split = blockIdx.x, splits = gridDim.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gq = lane / lpk, gl = lane - gq * lpk, gpw = 32 / lpk, ng = kDecWarps * gpw, grp = warp * gpw + gq;
    const int tile_keys = KT * ng;  // = kDecStageVecs / lpk
    const int per = (N + splits - 1) / splits, k0 = split * per, k1 = min(N, k0 + per);
    const int tiles = k1 > k0 ? (k1 - k0 + tile_keys - 1) / tile_keys : 0;
    const uint4 *Kg = reinterpret_cast<const uint4 *>(Kp + (size_t)unit * unit_elems);
    const uint4 *Vg = reinterpret_cast<const uint4 *>(Vp + (size_t)unit * unit_elems);

    // rows [k0 + t * tile_keys, ...) are contiguous in global memory: a stage is a straight copy of them
    auto issue = [&](int t) {
        if (t < tiles) {
            const size_t first = (size_t)(k0 + t * tile_keys) * lpk;
            const int nvec = min(tile_keys, k1 - (k0 + t * tile_keys)) * lpk;
            uint4 *sk = ring + (size_t)(t % kDecStages) * 2 * kDecStageVecs, *sv = sk + kDecStageVecs;
#pragma unroll
            for (int i = 0; i < KT; ++i) {
                const int v = i * kDecThreads + threadIdx.x;
                if (v < nvec) {
                    dec_cp_async16(sk + v, Kg + first + v);
                    dec_cp_async16(sv + v, Vg + first + v);
                }
            }
        }
        dec_cp_async_commit();  // one group per tile slot, empty or not, so that the wait below counts tiles
    };

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
#pragma unroll
    for (int t = 0; t < kDecStages - 1; ++t) issue(t);

    // Vector j * 256 + tid of a stage is slice gl of the key with slot j * ng + grp (ng * lpk = 256): every thread
    // consumes exactly the vectors it copied itself, so the ring needs no barrier, only the thread's own wait.
    for (int t = 0; t < tiles; ++t) {
        dec_cp_async_wait<kDecStages - 2>();  // this thread's copies of tile t have landed
        issue(t + kDecStages - 1);            // refills the stage this thread read in the previous round
        const uint4 *sk = ring + (size_t)(t % kDecStages) * 2 * kDecStageVecs + threadIdx.x, *sv = sk + kDecStageVecs;
        const int base = k0 + t * tile_keys;
        bool valid[KT];
        float s[KT][G];
#pragma unroll
        for (int j = 0; j < KT; ++j) {
            valid[j] = base + j * ng + grp < k1;
            float x[VE];
            RopeVec<T>::unpack(sk[j * kDecThreads], x);
#pragma unroll
            for (int h = 0; h < G; ++h) {
                float2 a = make_float2(0.f, 0.f);
#pragma unroll
                for (int i = 0; i < VE; i += 2) a = __ffma2_rn(make_float2(x[i], x[i + 1]), make_float2(qf[h][i], qf[h][i + 1]), a);
                s[j][h] = a.x + a.y;
            }
        }
        for (int off = lpk >> 1; off >= 1; off >>= 1) {
#pragma unroll
            for (int j = 0; j < KT; ++j)
#pragma unroll
                for (int h = 0; h < G; ++h) s[j][h] += __shfl_xor_sync(0xffffffffu, s[j][h], off);
        }
        bool moved = false;
        float mn[G];
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float mt = -INFINITY;
#pragma unroll
            for (int j = 0; j < KT; ++j) mt = fmaxf(mt, valid[j] ? s[j][h] : -INFINITY);
            mn[h] = fmaxf(m[h], mt);
            moved = moved || mn[h] > m[h];
        }
        if (__any_sync(0xffffffffu, moved)) {  // rare after the first tiles: a maximum moved, rescale the running output
#pragma unroll
            for (int h = 0; h < G; ++h) {
                const float corr = dec_scale(m[h], mn[h]);
                m[h] = mn[h];
                l[h] *= corr;
#pragma unroll
                for (int i = 0; i < VE; ++i) acc[h][i] *= corr;
            }
        }
#pragma unroll
        for (int j = 0; j < KT; ++j) {
            if (valid[j]) {  // a stage's unused rows hold stale bytes
                float x[VE];
                RopeVec<T>::unpack(sv[j * kDecThreads], x);
#pragma unroll
                for (int h = 0; h < G; ++h) {
                    const float p = dec_ex2(s[j][h] - m[h]);
                    l[h] += p;
#pragma unroll
                    for (int i = 0; i < VE; i += 2) {
                        const float2 r = __ffma2_rn(make_float2(p, p), make_float2(x[i], x[i + 1]), make_float2(acc[h][i], acc[h][i + 1]));
                        acc[h][i] = r.x;
                        acc[h][i + 1] = r.y;
                    }
                }
            }
        }
    }
    dec_cp_async_wait<0>();
    __syncthreads();  // the ring is free: its memory now carries the merge of the warps

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
