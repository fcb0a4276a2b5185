// CaP scoring (Sec. 3.3.1, Eq. 2) for bf16 pots whose head dimension the tcgen05 kernel does not take (any
// multiple of 16 up to 256, e.g. 96 or 256): the two launches of the fp32 scorer - row statistics, then
// column sums with the logits recomputed - with the products on warp-level m16n8k16 tensor-core tiles (fp32
// accumulation, so the logits are the same numbers the fp32 scorer sums).  Tiles are staged in shared memory
// with padded rows (fragment reads hit 32 different banks, see k_cap_self.cuh); a warp owns 16 query rows.
//   cap_row_stats_mma   : grid (ceil(M / 64), units, key splits); a block walks its share of the N keys in tiles
//                         of 64; every lane keeps the running (max, sum) of its two rows, so nothing crosses
//                         warps.  The key range is split so that small launches still fill the device; the
//                         partial pairs of a row are merged where they are used.
//   cap_column_sums_mma : grid (ceil(N / 64), units); a block keeps one 64-key tile and walks the query rows
//                         in tiles of 64; every lane accumulates its columns over all rows, the sums across
//                         lanes and warps are taken once at the end.
#pragma once
#include <cuda_bf16.h>

#include "common.cuh"
#include "k_cap_self.cuh"  // mma_bf16_16x8x16, self_stage, self_merge, kSelfPad

namespace ipotk {

constexpr int kMsWarps = 4;
constexpr int kMsRows = kMsWarps * 16;  // query rows per tile
constexpr int kMsKeys = 64;             // keys per tile

__host__ __device__ inline size_t mma_scorer_smem_bytes(int d) { return (size_t)(kMsRows + kMsKeys) * (d + kSelfPad) * 2; }

// S[16 rows of this warp][64 keys of the staged tile]: c[n][0], c[n][1] = row g, keys 8n + 2t, + 1; c[n][2], c[n][3] = row g + 8.
// The A fragments of a channel step are read once and used for all eight key tiles.
__device__ __forceinline__ void ms_tiles(float (&c)[kMsKeys / 8][4], const uint32_t *qa, const uint32_t *ks_base, int ksteps, int ws,
                                         int g, int t)
{
#pragma unroll
    for (int n = 0; n < kMsKeys / 8; ++n) c[n][0] = c[n][1] = c[n][2] = c[n][3] = 0.f;
    for (int ks = 0; ks < ksteps; ++ks) {
        const uint32_t a[4] = {qa[ks * 8 + t], qa[8 * ws + ks * 8 + t], qa[ks * 8 + 4 + t], qa[8 * ws + ks * 8 + 4 + t]};
#pragma unroll
        for (int n = 0; n < kMsKeys / 8; ++n) {
            const uint32_t *kr = ks_base + (n * 8 + g) * ws;
            mma_bf16_16x8x16(c[n], a, kr[ks * 8 + t], kr[ks * 8 + 4 + t]);
        }
    }
}

// part[(split * units + unit) * M + row] = (max logit in log2 units, sum_j 2^(x_j - max)) over the keys of the split
// (keys [split * per, (split + 1) * per), per a multiple of 64; an empty split writes (-inf, 0)).
__global__ void __launch_bounds__(kMsWarps * 32)
cap_row_stats_mma(const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ Kpot, float2 *__restrict__ part,
                  int M, int N, int d, size_t k_unit_stride, float scale_log2e, int per)
{
    extern __shared__ __align__(16) uint8_t ms_sm[];
    __nv_bfloat16 *Qs = reinterpret_cast<__nv_bfloat16 *>(ms_sm);
    __nv_bfloat16 *Ks = Qs + kMsRows * (d + kSelfPad);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int unit = blockIdx.y, row0 = blockIdx.x * kMsRows;
    const int ksteps = d / 16, ws = (d + kSelfPad) / 2;
    const int k_begin = blockIdx.z * per, k_end = min(N, k_begin + per);
    const __nv_bfloat16 *Ku = Kpot + (size_t)unit * k_unit_stride;
    self_stage(Qs, Q + (size_t)unit * M * d, row0, kMsRows, M, d);
    const uint32_t *qa = reinterpret_cast<const uint32_t *>(Qs) + (warp * 16 + g) * ws;
    float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
    for (int j0 = k_begin; j0 < k_end; j0 += kMsKeys) {
        if (j0 > k_begin) __syncthreads();  // the previous tile has been read
        self_stage(Ks, Ku, j0, kMsKeys, N, d);
        __syncthreads();
        const int nk = min(kMsKeys, k_end - j0);
        float cc[kMsKeys / 8][4];
        ms_tiles(cc, qa, reinterpret_cast<const uint32_t *>(Ks), ksteps, ws, g, t);
#pragma unroll
        for (int n = 0; n < kMsKeys / 8; ++n) {
            const int n0 = n * 8;
            const float (&c)[4] = cc[n];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const float x0 = c[2 * h] * scale_log2e, x1 = c[2 * h + 1] * scale_log2e;
                const bool v0 = n0 + 2 * t < nk, v1 = n0 + 2 * t + 1 < nk;
                const float tm = fmaxf(v0 ? x0 : -INFINITY, v1 ? x1 : -INFINITY);
                if (tm > -INFINITY) self_merge(m[h], l[h], tm, (v0 ? exp2f(x0 - tm) : 0.f) + (v1 ? exp2f(x1 - tm) : 0.f));
            }
        }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
#pragma unroll
        for (int off = 1; off <= 2; off <<= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, m[h], off), l2 = __shfl_xor_sync(0xffffffffu, l[h], off);
            self_merge(m[h], l[h], m2, l2);
        }
        const int row = row0 + warp * 16 + g + 8 * h;
        if (t == 0 && row < M) part[((size_t)blockIdx.z * gridDim.y + unit) * M + row] = make_float2(m[h], l[h]);
    }
}

// The row's (max, 1 / sum) from its nsplit partial pairs and, if given, the extra pair (the CaP keys' share).
__device__ __forceinline__ float2 ms_row_weight(const float2 *__restrict__ part, const float2 *__restrict__ extra, int nsplit,
                                                size_t split_stride, size_t idx)
{
    float m = -INFINITY, l = 0.f;
    for (int s = 0; s < nsplit; ++s) {
        const float2 p = part[(size_t)s * split_stride + idx];
        self_merge(m, l, p.x, p.y);
    }
    if (extra) {
        const float2 e = extra[idx];
        self_merge(m, l, e.x, e.y);
    }
    return make_float2(m, 1.f / l);
}

// scores[unit][j] = sum_i 2^(x_ij - max_i) / denom_i for the 64 keys of the block.
__global__ void __launch_bounds__(kMsWarps * 32)
cap_column_sums_mma(const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ Kpot, const float2 *__restrict__ part,
                    const float2 *__restrict__ extra, int nsplit, float *__restrict__ scores, int M, int N, int d,
                    size_t k_unit_stride, float scale_log2e)
{
    extern __shared__ __align__(16) uint8_t ms_sm[];
    __nv_bfloat16 *Qs = reinterpret_cast<__nv_bfloat16 *>(ms_sm);
    __nv_bfloat16 *Ks = Qs + kMsRows * (d + kSelfPad);
    __shared__ float colsum[kMsWarps][kMsKeys];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int unit = blockIdx.y, j0 = blockIdx.x * kMsKeys;
    const int ksteps = d / 16, ws = (d + kSelfPad) / 2;
    self_stage(Ks, Kpot + (size_t)unit * k_unit_stride, j0, kMsKeys, N, d);
    const uint32_t *qa = reinterpret_cast<const uint32_t *>(Qs) + (warp * 16 + g) * ws;
    float col[kMsKeys / 8][2];  // this lane's columns 8 n + 2t, + 1 summed over its rows
#pragma unroll
    for (int n = 0; n < kMsKeys / 8; ++n) col[n][0] = col[n][1] = 0.f;
    for (int i0 = 0; i0 < M; i0 += kMsRows) {
        if (i0 > 0) __syncthreads();
        self_stage(Qs, Q + (size_t)unit * M * d, i0, kMsRows, M, d);
        __syncthreads();
        const int r0 = i0 + warp * 16 + g, r1 = r0 + 8;
        const size_t sstride = (size_t)gridDim.y * M;
        const float2 s0 = r0 < M ? ms_row_weight(part, extra, nsplit, sstride, (size_t)unit * M + r0) : make_float2(0.f, 0.f);
        const float2 s1 = r1 < M ? ms_row_weight(part, extra, nsplit, sstride, (size_t)unit * M + r1) : make_float2(0.f, 0.f);  // rows beyond M weigh nothing
        float cc[kMsKeys / 8][4];
        ms_tiles(cc, qa, reinterpret_cast<const uint32_t *>(Ks), ksteps, ws, g, t);
#pragma unroll
        for (int n = 0; n < kMsKeys / 8; ++n) {
            const float (&c)[4] = cc[n];
            col[n][0] += exp2f(c[0] * scale_log2e - s0.x) * s0.y + exp2f(c[2] * scale_log2e - s1.x) * s1.y;
            col[n][1] += exp2f(c[1] * scale_log2e - s0.x) * s0.y + exp2f(c[3] * scale_log2e - s1.x) * s1.y;
        }
    }
    // lanes with the same t hold the same columns: add the eight row groups, then the four warps
#pragma unroll
    for (int n = 0; n < kMsKeys / 8; ++n) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float v = col[n][h];
            v += __shfl_xor_sync(0xffffffffu, v, 4);
            v += __shfl_xor_sync(0xffffffffu, v, 8);
            v += __shfl_xor_sync(0xffffffffu, v, 16);
            if (g == 0) colsum[warp][n * 8 + 2 * t + h] = v;
        }
    }
    __syncthreads();
    if (threadIdx.x < kMsKeys && j0 + threadIdx.x < N)
        scores[(size_t)unit * N + j0 + threadIdx.x] =
            (colsum[0][threadIdx.x] + colsum[1][threadIdx.x]) + (colsum[2][threadIdx.x] + colsum[3][threadIdx.x]);
}

}  // namespace ipotk
