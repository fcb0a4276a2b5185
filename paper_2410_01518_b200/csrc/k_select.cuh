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
#pragma once
#include "common.cuh"

namespace ipotk {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;

struct SelShared {
    uint32_t hist[256];
    int wtot[2][kSelWarps];
    uint32_t bin;
    int remaining;
    int bin_count;
};

// k-th largest key (k >= 1) among keys[0..N): returns the key value, how many
// keys equal to it must be taken (need_eq >= 1) and how many such keys exist.
__device__ inline void block_radix_select(const uint32_t *keys, int N, int k, SelShared &sh,
                                          uint32_t &tau, int &need_eq, int &count_eq)
{
    uint32_t prefix = 0, mask = 0;
    int remaining = k;
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (threadIdx.x < 256) sh.hist[threadIdx.x] = 0;
        __syncthreads();
        for (int j = threadIdx.x; j < N; j += blockDim.x) {
            const uint32_t key = keys[j];
            if ((key & mask) == prefix) atomicAdd(&sh.hist[(key >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            // lane l owns the 8 bins 255 - 8l ... 248 - 8l (descending key order)
            const int lane = threadIdx.x;
            uint32_t c[8], tot = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) { c[i] = sh.hist[255 - (8 * lane + i)]; tot += c[i]; }
            uint32_t inc = tot;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t v = __shfl_up_sync(0xffffffffu, inc, off);
                if (lane >= off) inc += v;
            }
            uint32_t run = inc - tot;  // keys in bins above this lane's bins
            if (run < (uint32_t)remaining && (uint32_t)remaining <= inc) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (run + c[i] >= (uint32_t)remaining) {
                        sh.bin = 255 - (8 * lane + i);
                        sh.remaining = remaining - (int)run;
                        sh.bin_count = (int)c[i];
                        break;
                    }
                    run += c[i];
                }
            }
        }
        __syncthreads();
        prefix |= sh.bin << shift;
        mask |= 255u << shift;
        remaining = sh.remaining;
    }
    tau = prefix;
    need_eq = remaining;
    count_eq = sh.bin_count;
    __syncthreads();
}

// Exclusive prefix count of `flag` over the block in thread order; `total` = block sum.
__device__ __forceinline__ int block_prefix_count(bool flag, SelShared &sh, int parity, int &total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t b = __ballot_sync(0xffffffffu, flag);
    const int in_warp = __popc(b & ((1u << lane) - 1u));
    if (lane == 0) sh.wtot[parity][warp] = __popc(b);
    __syncthreads();
    int v = (lane < kSelWarps) ? sh.wtot[parity][lane] : 0;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, v, off);
        if (lane >= off) v += t;
    }
    total = __shfl_sync(0xffffffffu, v, 31);
    const int before = __shfl_sync(0xffffffffu, v, (warp + 31) & 31);
    return in_warp + (warp == 0 ? 0 : before);
}

// Ordered sweep: slot j is taken iff key > tau, or key == tau and it is among the
// first need_eq such slots.  taken(j, pos) is called for every taken slot with its
// rank pos among the taken ones; every(j, is_taken) for every slot.
template <typename Taken, typename Every>
__device__ inline void block_ordered_sweep(const uint32_t *keys, int N, uint32_t tau, int need_eq,
                                           int count_eq, SelShared &sh, Taken taken, Every every)
{
    const bool rank_ties = need_eq < count_eq;
    int base_eq = 0, base_out = 0, parity = 0;
    for (int j0 = 0; j0 < N; j0 += blockDim.x) {
        const int j = j0 + threadIdx.x;
        const bool valid = j < N;
        const uint32_t key = valid ? keys[j] : 0u;
        const bool gt = valid && key > tau;
        const bool eq = valid && key == tau;
        bool sel = gt || eq;
        if (rank_ties) {
            int tot;
            const int r = base_eq + block_prefix_count(eq, sh, parity, tot);
            parity ^= 1;
            base_eq += tot;
            sel = gt || (eq && r < need_eq);
        }
        int tot;
        const int pos = base_out + block_prefix_count(sel, sh, parity, tot);
        parity ^= 1;
        base_out += tot;
        if (valid) every(j, sel);
        if (sel) taken(j, pos);
    }
}

struct SelNoTaken { __device__ void operator()(int, int) const {} };
struct SelNoEvery { __device__ void operator()(int, bool) const {} };
struct SelWriteMask {
    uint8_t *m;
    __device__ void operator()(int j, bool s) const { m[j] = s ? 1 : 0; }
};
struct SelWriteIndex {
    int32_t *out;
    int keep;
    int *status;
    __device__ void operator()(int j, int pos) const
    {
        if (pos < keep) out[pos] = j;
        else set_status(status, kStatusBounds);
    }
};

// grid (batch).  mask[b][j] = 1 iff slot j is one of the T most novel slots of stream b.
__global__ void __launch_bounds__(kSelThreads)
nuc_mask_kernel(const float *__restrict__ aux, uint8_t *__restrict__ mask, int N, int T)
{
    extern __shared__ __align__(16) uint32_t sel_keys[];
    __shared__ SelShared sh;
    const float *a = aux + (size_t)blockIdx.x * N;
    for (int j = threadIdx.x; j < N; j += blockDim.x) sel_keys[j] = order_key(a[j]);
    __syncthreads();
    uint32_t tau;
    int need_eq, count_eq;
    block_radix_select(sel_keys, N, T, sh, tau, need_eq, count_eq);
    block_ordered_sweep(sel_keys, N, tau, need_eq, count_eq, sh, SelNoTaken{},
                        SelWriteMask{mask + (size_t)blockIdx.x * N});
}

// grid (units).  scores: `parts` partial score arrays of [units][N] each, `part_stride`
// floats apart, added in index order.  mask may be NULL (T == 0).
__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float *__restrict__ scores, int parts, size_t part_stride,
              const uint8_t *__restrict__ mask, int32_t *__restrict__ idx, float *__restrict__ summed,
              int N, int keep, int Hkv, int batch, int *status)
{
    extern __shared__ __align__(16) uint32_t sel_keys[];
    __shared__ SelShared sh;
    const int unit = blockIdx.x;
    const int b = (unit / Hkv) % batch;
    const float *u = scores + (size_t)unit * N;
    const uint8_t *m = mask ? mask + (size_t)b * N : nullptr;
    for (int j = threadIdx.x; j < N; j += blockDim.x) {
        float s = u[j];
        for (int p = 1; p < parts; ++p) s += u[(size_t)p * part_stride + j];
        if (summed) summed[(size_t)unit * N + j] = s;
        // a reserved slot outranks every score: finite scores map below 0xFF800000
        sel_keys[j] = (m && m[j]) ? 0xFFFFFFFFu : order_key(s);
    }
    __syncthreads();
    uint32_t tau;
    int need_eq, count_eq;
    block_radix_select(sel_keys, N, keep, sh, tau, need_eq, count_eq);
    block_ordered_sweep(sel_keys, N, tau, need_eq, count_eq, sh,
                        SelWriteIndex{idx + (size_t)unit * keep, keep, status}, SelNoEvery{});
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
