// Rankings of the cycle (Sec. 3.3.3, Appendix B "Combine NuC and CaP" and "Final
// Token Selection"):
//   nuc_mask_kernel   : per stream, mark the T slots with the largest novelty;
//   select_kernel     : per unit, give the marked slots the highest possible
//                       key, take the top `keep` keys, emit the survivors'
//                       slot numbers in ascending order.
// Both are an exact radix select on an order-preserving 32-bit image of the
// fp32 value (4 passes of 8 bits, most significant first) followed by one
// ordered sweep; among equal keys the lower slot wins, so the result is a pure
// function of the score bits.
//
// One block per problem.  A thread keeps 16 (pot sizes above 16384: 32) consecutive
// slots' keys in registers from the first load to the last store, and the block has
// only as many threads as that takes (256 for a pot of 4096): the per-thread work of
// a pass (histogram scan, barriers) is then shared by 16 keys, which is what the
// instruction count - the bound of this kernel - is made of.  Slots beyond N carry key
// 0, which no score maps to, and are never taken.
#pragma once
#include "common.cuh"

namespace ipotk {

constexpr int kSelMaxWarps = 32;

struct SelShared {
    __align__(16) uint32_t hist[256];
    uint32_t wtot[2][kSelMaxWarps];
    uint32_t bin;
    int remaining;
};

// Exclusive prefix sum of v over the block in thread order; `total` = block sum.  One barrier; consecutive
// calls alternate `parity` so that a warp that runs ahead does not overwrite totals still being read.
template <int kThreads>
__device__ __forceinline__ uint32_t block_scan_exclusive(uint32_t v, SelShared &sh, int parity, uint32_t &total)
{
    constexpr int kWarps = kThreads / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += t;
    }
    if (lane == 31) sh.wtot[parity][warp] = inc;
    __syncthreads();
    uint32_t w = lane < kWarps ? sh.wtot[parity][lane] : 0u;
#pragma unroll
    for (int off = 1; off < kWarps; off <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, w, off);
        if (lane >= off) w += t;
    }
    total = __shfl_sync(0xffffffffu, w, kWarps - 1);
    const uint32_t before = __shfl_sync(0xffffffffu, w, (warp + 31) & 31);
    return (warp == 0 ? 0u : before) + inc - v;
}

// k-th largest (k >= 1) of the block's keys: returns the key value and how many keys equal to it
// must be taken (need_eq >= 1).  sh.hist must be zero on entry and is zero again on exit.
template <int kThreads, int kKpt>
__device__ __forceinline__ void block_radix_select(const uint32_t (&key)[kKpt], int k, SelShared &sh,
                                                   uint32_t &tau, int &need_eq)
{
    uint32_t prefix = 0, mask = 0;
    int remaining = k;
    const int lane = threadIdx.x & 31;
#pragma unroll 1
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (shift == 24) {
            // leading byte (sign and exponent): the scores of a problem sit within a few binades, so a thread's keys -
            // often a warp's - share it; they are counted in registers and leave as one update
            const uint32_t d0 = key[0] >> 24;
            uint32_t cnt = 0;
#pragma unroll
            for (int i = 0; i < kKpt; ++i) cnt += (key[i] >> 24) == d0 ? 1u : 0u;
            if (__all_sync(0xffffffffu, d0 == __shfl_sync(0xffffffffu, d0, 0))) {
                const uint32_t tot = __reduce_add_sync(0xffffffffu, cnt);
                if (lane == 0) atomicAdd(&sh.hist[d0], tot);
            } else {
                atomicAdd(&sh.hist[d0], cnt);
            }
#pragma unroll
            for (int i = 1; i < kKpt; ++i)
                if ((key[i] >> 24) != d0) atomicAdd(&sh.hist[key[i] >> 24], 1u);
        } else {
#pragma unroll
            for (int i = 0; i < kKpt; ++i)
                if ((key[i] & mask) == prefix) atomicAdd(&sh.hist[(key[i] >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            // lane l owns the 8 bins 255 - 8l ... 248 - 8l (descending key order) and clears them for the next pass
            uint4 *h4 = reinterpret_cast<uint4 *>(sh.hist) + (62 - 2 * lane);
            const uint4 lo = h4[0], hi = h4[1];
            h4[0] = make_uint4(0u, 0u, 0u, 0u);
            h4[1] = make_uint4(0u, 0u, 0u, 0u);
            const uint32_t c[8] = {hi.w, hi.z, hi.y, hi.x, lo.w, lo.z, lo.y, lo.x};
            const uint32_t tot = ((c[0] + c[1]) + (c[2] + c[3])) + ((c[4] + c[5]) + (c[6] + c[7]));
            uint32_t inc = tot;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t v = __shfl_up_sync(0xffffffffu, inc, off);
                if (lane >= off) inc += v;
            }
            uint32_t run = inc - tot;  // keys in the bins above this lane's
            if (run < (uint32_t)remaining && (uint32_t)remaining <= inc) {
                int found = 7;
#pragma unroll
                for (int i = 6; i >= 0; --i) {  // the first bin that reaches `remaining`
                    uint32_t upto = run;
#pragma unroll
                    for (int e = 0; e <= i; ++e) upto += c[e];
                    if (upto >= (uint32_t)remaining) found = i;
                }
#pragma unroll
                for (int e = 0; e < 7; ++e) run += e < found ? c[e] : 0u;
                sh.bin = 255u - (8u * lane + found);
                sh.remaining = remaining - (int)run;
            }
        }
        __syncthreads();
        prefix |= sh.bin << shift;
        mask |= 255u << shift;
        remaining = sh.remaining;
    }
    tau = prefix;
    need_eq = remaining;
}

// Larger and equal keys in the slots below this thread's, in one block scan (16 bits each: a block has at
// most 32768 slots); `total` = the same counts over the block.
template <int kThreads, int kKpt>
__device__ __forceinline__ uint32_t block_count_before(const uint32_t (&key)[kKpt], uint32_t tau, SelShared &sh, uint32_t &total)
{
    uint32_t mine = 0;
#pragma unroll
    for (int i = 0; i < kKpt; ++i) mine += (key[i] > tau ? 1u : 0u) + (key[i] == tau ? 0x10000u : 0u);
    return block_scan_exclusive<kThreads>(mine, sh, 0, total);
}
// Ordered sweep: slot j is taken iff key > tau, or key == tau and it is among the first need_eq such
// slots.  taken(j, pos) is called for every taken slot with its rank pos among the taken ones;
// every(i, is_taken) for each of the thread's slots i < kKpt.  `before` = block_count_before().
template <int kThreads, int kKpt, typename Taken, typename Every>
__device__ __forceinline__ void block_ordered_sweep(const uint32_t (&key)[kKpt], int slot0, uint32_t tau, int need_eq,
                                                    uint32_t before, Taken taken, Every every)
{
    int gt_before = (int)(before & 0xFFFFu), eq_before = (int)(before >> 16);
#pragma unroll
    for (int i = 0; i < kKpt; ++i) {
        const bool gt = key[i] > tau, eq = key[i] == tau;
        const bool sel = gt || (eq && eq_before < need_eq);
        every(i, sel);
        if (sel) taken(slot0 + i, gt_before + min(eq_before, need_eq));
        gt_before += gt;
        eq_before += eq;
    }
}

struct SelNoTaken { __device__ void operator()(int, int) const {} };
struct SelNoEvery { __device__ void operator()(int, bool) const {} };
constexpr int kSelStage = 4096;   // survivors staged in shared memory per round of the index output
struct SelStageIndex {            // positions [base, base + kSelStage) go to the stage, the rest to another round
    int32_t *stage;
    int base;
    __device__ void operator()(int j, int pos) const
    {
        if ((unsigned)(pos - base) < (unsigned)kSelStage) stage[pos - base] = j;
    }
};
struct SelPackMask {  // byte i of the thread's mask bytes, four to a word
    uint32_t *packed;
    __device__ void operator()(int i, bool s) const { packed[i >> 2] |= (s ? 1u : 0u) << (8 * (i & 3)); }
};

// grid (batch).  mask[b][j] = 1 iff slot j is one of the T most novel slots of stream b.
template <int kThreads, int kKpt>
__global__ void __launch_bounds__(kThreads)
nuc_mask_kernel(const float *__restrict__ aux, uint8_t *__restrict__ mask, int N, int T)
{
    __shared__ SelShared sh;
    const float *a = aux + (size_t)blockIdx.x * N;
    uint8_t *m = mask + (size_t)blockIdx.x * N;
    const int slot0 = threadIdx.x * kKpt;
    if (threadIdx.x < 256) sh.hist[threadIdx.x] = 0;
    uint32_t key[kKpt];
    const bool vec = (N & 15) == 0 && slot0 + kKpt <= N;   // rows of N floats (and of N bytes) stay 16-byte aligned
    if (vec) {
#pragma unroll
        for (int i = 0; i < kKpt; i += 4) {
            const float4 v = *reinterpret_cast<const float4 *>(a + slot0 + i);
            key[i] = order_key(v.x);
            key[i + 1] = order_key(v.y);
            key[i + 2] = order_key(v.z);
            key[i + 3] = order_key(v.w);
        }
    } else {
#pragma unroll
        for (int i = 0; i < kKpt; ++i) key[i] = slot0 + i < N ? order_key(a[slot0 + i]) : 0u;
    }
    __syncthreads();
    uint32_t tau;
    int need_eq;
    block_radix_select<kThreads, kKpt>(key, T, sh, tau, need_eq);
    uint32_t packed[kKpt / 4];
#pragma unroll
    for (int i = 0; i < kKpt / 4; ++i) packed[i] = 0;
    uint32_t total;
    const uint32_t before = block_count_before<kThreads, kKpt>(key, tau, sh, total);
    block_ordered_sweep<kThreads, kKpt>(key, slot0, tau, need_eq, before, SelNoTaken{}, SelPackMask{packed});
    if (vec) {
#pragma unroll
        for (int i = 0; i < kKpt / 4; i += 4)
            *reinterpret_cast<uint4 *>(m + slot0 + 4 * i) = make_uint4(packed[i], packed[i + 1], packed[i + 2], packed[i + 3]);
    } else {
#pragma unroll
        for (int i = 0; i < kKpt; ++i)
            if (slot0 + i < N) m[slot0 + i] = (uint8_t)((packed[i >> 2] >> (8 * (i & 3))) & 1u);
    }
}

// grid (units).  scores: `parts` partial score arrays of [units][N] each, `part_stride`
// floats apart, added in index order.  mask may be NULL (T == 0).  The survivors' slot numbers
// are put in order in shared memory and leave in 16-byte stores.
template <int kThreads, int kKpt>
__global__ void __launch_bounds__(kThreads)
select_kernel(const float *__restrict__ scores, int parts, size_t part_stride,
              const uint8_t *__restrict__ mask, int32_t *__restrict__ idx, float *__restrict__ summed,
              int N, int keep, int Hkv, int batch, int *status)
{
    __shared__ SelShared sh;
    __shared__ __align__(16) int32_t stage[kSelStage];
    const int unit = blockIdx.x;
    const int b = (unit / Hkv) % batch;
    const float *u = scores + (size_t)unit * N;
    const uint8_t *m = mask ? mask + (size_t)b * N : nullptr;
    const int slot0 = threadIdx.x * kKpt;
    // the compaction may be made resident now; it waits for this grid's end before it reads an index
    asm volatile("griddepcontrol.launch_dependents;");
    if (threadIdx.x < 256) sh.hist[threadIdx.x] = 0;
    uint32_t key[kKpt];
    // a reserved slot outranks every score: finite scores map below 0xFF800000
    if ((N & 15) == 0 && (part_stride & 3) == 0 && slot0 + kKpt <= N) {
        float4 s[kKpt / 4];
        uint32_t r[kKpt / 4];
#pragma unroll
        for (int i = 0; i < kKpt / 4; ++i) s[i] = *reinterpret_cast<const float4 *>(u + slot0 + 4 * i);   // all loads in flight together
#pragma unroll
        for (int i = 0; i < kKpt / 4; ++i) r[i] = m ? *reinterpret_cast<const uint32_t *>(m + slot0 + 4 * i) : 0u;
        if (parts > 1) {
#pragma unroll 1
            for (int p = 1; p < parts; ++p) {
#pragma unroll
                for (int i = 0; i < kKpt / 4; ++i) {
                    const float4 t = *reinterpret_cast<const float4 *>(u + (size_t)p * part_stride + slot0 + 4 * i);
                    s[i].x += t.x;
                    s[i].y += t.y;
                    s[i].z += t.z;
                    s[i].w += t.w;
                }
            }
            if (summed) {
#pragma unroll
                for (int i = 0; i < kKpt / 4; ++i) *reinterpret_cast<float4 *>(summed + (size_t)unit * N + slot0 + 4 * i) = s[i];
            }
        }
#pragma unroll
        for (int i = 0; i < kKpt / 4; ++i) {
            key[4 * i] = (r[i] & 0xFFu) ? 0xFFFFFFFFu : order_key(s[i].x);
            key[4 * i + 1] = (r[i] & 0xFF00u) ? 0xFFFFFFFFu : order_key(s[i].y);
            key[4 * i + 2] = (r[i] & 0xFF0000u) ? 0xFFFFFFFFu : order_key(s[i].z);
            key[4 * i + 3] = (r[i] & 0xFF000000u) ? 0xFFFFFFFFu : order_key(s[i].w);
        }
    } else {
#pragma unroll
        for (int i = 0; i < kKpt; ++i) {
            const int j = slot0 + i;
            key[i] = 0u;
            if (j < N) {
                float s = u[j];
#pragma unroll 1
                for (int p = 1; p < parts; ++p) s += u[(size_t)p * part_stride + j];
                if (summed && parts > 1) summed[(size_t)unit * N + j] = s;
                key[i] = (m && m[j]) ? 0xFFFFFFFFu : order_key(s);
            }
        }
    }
    __syncthreads();
    uint32_t tau;
    int need_eq;
    block_radix_select<kThreads, kKpt>(key, keep, sh, tau, need_eq);
    uint32_t total;
    const uint32_t before = block_count_before<kThreads, kKpt>(key, tau, sh, total);
    const int taken = (int)(total & 0xFFFFu) + min((int)(total >> 16), need_eq);
    if (taken != keep && threadIdx.x == 0) set_status(status, kStatusBounds);
    int32_t *out = idx + (size_t)unit * keep;
    for (int base = 0; base < keep; base += kSelStage) {
        block_ordered_sweep<kThreads, kKpt>(key, slot0, tau, need_eq, before, SelStageIndex{stage, base}, SelNoEvery{});
        __syncthreads();
        const int n = min(kSelStage, min(keep, taken) - base);
        if ((keep & 3) == 0) {
            for (int i = 4 * threadIdx.x; i < n; i += 4 * kThreads) {
                if (i + 4 <= n) *reinterpret_cast<int4 *>(out + base + i) = *reinterpret_cast<const int4 *>(stage + i);
                else
                    for (int e = i; e < n; ++e) out[base + e] = stage[e];
            }
        } else {
            for (int i = threadIdx.x; i < n; i += kThreads) out[base + i] = stage[i];
        }
        if (base + kSelStage < keep) __syncthreads();
    }
}

// Launch shapes: the smallest block whose threads hold N slots at 16 a thread (32 above 16384 slots).
#define IPOT_SEL_DISPATCH(kernel, blocks, stream, N, ...)                                        \
    do {                                                                                         \
        if ((N) <= 4096) kernel<256, 16><<<(blocks), 256, 0, (stream)>>>(__VA_ARGS__);           \
        else if ((N) <= 8192) kernel<512, 16><<<(blocks), 512, 0, (stream)>>>(__VA_ARGS__);      \
        else if ((N) <= 16384) kernel<1024, 16><<<(blocks), 1024, 0, (stream)>>>(__VA_ARGS__);   \
        else kernel<1024, 32><<<(blocks), 1024, 0, (stream)>>>(__VA_ARGS__);                     \
    } while (0)

inline void launch_nuc_mask(int blocks, cudaStream_t st, const float *aux, uint8_t *mask, int N, int T)
{
    IPOT_SEL_DISPATCH(nuc_mask_kernel, blocks, st, N, aux, mask, N, T);
}
inline void launch_select(int blocks, cudaStream_t st, const float *scores, int parts, size_t part_stride, const uint8_t *mask,
                          int32_t *idx, float *summed, int N, int keep, int Hkv, int batch, int *status)
{
    IPOT_SEL_DISPATCH(select_kernel, blocks, st, N, scores, parts, part_stride, mask, idx, summed, N, keep, Hkv, batch, status);
}

// summed[i] = parts[0][i] + parts[1][i] + ... in index order (the order select_kernel uses).
__global__ void sum_parts_kernel(const float *__restrict__ scores, int parts, size_t part_stride,
                                 float *__restrict__ summed, size_t n)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float s = scores[i];
    for (int p = 1; p < parts; ++p) s += scores[(size_t)p * part_stride + i];
    summed[i] = s;
}

}  // namespace ipotk
