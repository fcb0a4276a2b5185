// CaP scoring with plain fp32 FMAs (Sec. 3.3.1, Eq. 2): any supported shape,
// f32 or bf16 storage.  Two launches per cycle:
//   cap_row_stats  : per query row, the maximum logit and the reciprocal of the
//                    softmax denominator over the N pot keys;  the same kernel,
//                    run over the CaP's own keys with a causal limit, gives the
//                    share of the denominator that Appendix B's listing adds
//                    (CaP queries also attend to the CaP keys before them);
//   cap_column_sums: recomputes the logits per 64-key slab and adds
//                    exp(s - max) / denominator over all query rows of the unit.
// The M x N probability matrix lives only in registers.  Logits are kept in
// log2 units (s * log2(e) / sqrt(d)) so that exp() is one ex2.
#pragma once
#include "common.cuh"

namespace ipotk {

constexpr int kSimtRows = 32;  // query rows per tile
constexpr int kSimtKeys = 64;  // keys per tile
constexpr int kSimtThreads = 256;

__host__ __device__ inline size_t simt_smem_bytes(int d)
{
    return (size_t)(kSimtRows + kSimtKeys) * (size_t)(d + 4) * sizeof(float);
}

// Rows [row0, row0 + rows) of a [limit][d] matrix -> smem floats, row stride d + 4;
// rows at or beyond `limit` become zeros.
template <typename T>
__device__ __forceinline__ void stage_rows(float *dst, const T *src, int row0, int rows, int limit, int d)
{
    constexpr int VE = Vec16<T>::kElems;
    const int vpr = d / VE;
    const int ds = d + 4;
    for (int v = threadIdx.x; v < rows * vpr; v += kSimtThreads) {
        const int r = v / vpr, c = (v - r * vpr) * VE;
        float f[VE];
        if (row0 + r < limit) {
            Vec16<T>::load(src + (size_t)(row0 + r) * d + c, f);
        } else {
#pragma unroll
            for (int i = 0; i < VE; ++i) f[i] = 0.f;
        }
#pragma unroll
        for (int i = 0; i < VE; i += 4)
            *reinterpret_cast<float4 *>(dst + r * ds + c + i) = make_float4(f[i], f[i + 1], f[i + 2], f[i + 3]);
    }
}

// acc[a][b] = q(ty + 16a) . k(tx + 16b)
__device__ __forceinline__ void tile_dots(const float *Qs, const float *Ks, int d, int tx, int ty,
                                          float acc[2][4])
{
    const int ds = d + 4;
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
    for (int c = 0; c < d; c += 4) {
        float4 q[2], k[4];
#pragma unroll
        for (int a = 0; a < 2; ++a) q[a] = *reinterpret_cast<const float4 *>(Qs + (ty + 16 * a) * ds + c);
#pragma unroll
        for (int b = 0; b < 4; ++b) k[b] = *reinterpret_cast<const float4 *>(Ks + (tx + 16 * b) * ds + c);
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                acc[a][b] = fmaf(q[a].x, k[b].x, acc[a][b]);
                acc[a][b] = fmaf(q[a].y, k[b].y, acc[a][b]);
                acc[a][b] = fmaf(q[a].z, k[b].z, acc[a][b]);
                acc[a][b] = fmaf(q[a].w, k[b].w, acc[a][b]);
            }
    }
}

__device__ __forceinline__ void merge_stats(float &m, float &l, float m2, float l2)
{
    const float mn = fmaxf(m, m2);
    const float a = (m == -INFINITY) ? 0.f : l * exp2f(m - mn);
    const float b = (m2 == -INFINITY) ? 0.f : l2 * exp2f(m2 - mn);
    m = mn;
    l = a + b;
}

// grid (ceil(M / 32), units).  Row statistics over the keys Kpot[unit][0..N): (max logit in log2 units, sum_j 2^(x_j - max)).
//   causal_P > 0 : row r only sees the keys 0 .. r % causal_P (the CaP keys up to the row's own position);
//   extra        : if not NULL, (max, sum) pairs [unit][M] merged into the row's statistics first;
//   reciprocal   : store 1 / sum instead of the sum (what cap_column_sums multiplies by).
template <typename T>
__global__ void __launch_bounds__(kSimtThreads)
cap_row_stats(const T *__restrict__ Q, const T *__restrict__ Kpot, float2 *__restrict__ stats,
              int M, int N, int d, size_t k_unit_stride, float scale_log2e,
              const float2 *__restrict__ extra, int causal_P, int reciprocal)
{
    extern __shared__ __align__(16) float simt_sm[];
    float *Qs = simt_sm, *Ks = simt_sm + kSimtRows * (d + 4);
    const int unit = blockIdx.y, i0 = blockIdx.x * kSimtRows;
    const T *Qu = Q + (size_t)unit * M * d;
    const T *Ku = Kpot + (size_t)unit * k_unit_stride;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;

    stage_rows(Qs, Qu, i0, kSimtRows, M, d);
    float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
    int lim[2];  // keys this thread's rows may see
#pragma unroll
    for (int a = 0; a < 2; ++a) lim[a] = causal_P > 0 ? min(N, (i0 + ty + 16 * a) % causal_P + 1) : N;
    for (int j0 = 0; j0 < N; j0 += kSimtKeys) {
        __syncthreads();
        stage_rows(Ks, Ku, j0, kSimtKeys, N, d);
        __syncthreads();
        float acc[2][4];
        tile_dots(Qs, Ks, d, tx, ty, acc);
#pragma unroll
        for (int a = 0; a < 2; ++a) {
            float tm = -INFINITY;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                acc[a][b] *= scale_log2e;
                if (j0 + tx + 16 * b < lim[a]) tm = fmaxf(tm, acc[a][b]);
            }
            if (tm > -INFINITY) {
                float tl = 0.f;
#pragma unroll
                for (int b = 0; b < 4; ++b)
                    if (j0 + tx + 16 * b < lim[a]) tl += exp2f(acc[a][b] - tm);
                merge_stats(m[a], l[a], tm, tl);
            }
        }
    }
#pragma unroll
    for (int a = 0; a < 2; ++a) {
#pragma unroll
        for (int off = 8; off >= 1; off >>= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, m[a], off);
            const float l2 = __shfl_xor_sync(0xffffffffu, l[a], off);
            merge_stats(m[a], l[a], m2, l2);
        }
        const int row = i0 + ty + 16 * a;
        if (tx == 0 && row < M) {
            if (extra) {
                const float2 e = extra[(size_t)unit * M + row];
                merge_stats(m[a], l[a], e.x, e.y);
            }
            stats[(size_t)unit * M + row] = make_float2(m[a], reciprocal ? 1.f / l[a] : l[a]);
        }
    }
}

// grid (ceil(N / 64), units).  scores[unit][j] = sum_i 2^(x_ij - max_i) / denom_i.
template <typename T>
__global__ void __launch_bounds__(kSimtThreads)
cap_column_sums(const T *__restrict__ Q, const T *__restrict__ Kpot, const float2 *__restrict__ stats,
                float *__restrict__ scores, int M, int N, int d, size_t k_unit_stride, float scale_log2e)
{
    extern __shared__ __align__(16) float simt_sm[];
    float *Qs = simt_sm, *Ks = simt_sm + kSimtRows * (d + 4);
    const int unit = blockIdx.y, j0 = blockIdx.x * kSimtKeys;
    const T *Qu = Q + (size_t)unit * M * d;
    const T *Ku = Kpot + (size_t)unit * k_unit_stride;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;

    stage_rows(Ks, Ku, j0, kSimtKeys, N, d);
    float col[4] = {0.f, 0.f, 0.f, 0.f};
    for (int i0 = 0; i0 < M; i0 += kSimtRows) {
        __syncthreads();
        stage_rows(Qs, Qu, i0, kSimtRows, M, d);
        __syncthreads();
        float acc[2][4];
        tile_dots(Qs, Ks, d, tx, ty, acc);
#pragma unroll
        for (int a = 0; a < 2; ++a) {
            const int row = i0 + ty + 16 * a;
            if (row < M) {
                const float2 st = stats[(size_t)unit * M + row];
#pragma unroll
                for (int b = 0; b < 4; ++b) col[b] += exp2f(acc[a][b] * scale_log2e - st.x) * st.y;
            }
        }
    }
    __syncthreads();
    float *red = simt_sm;  // [16][64], reuses the Q tile area (32 * (d + 4) >= 1024 floats for d >= 28)
#pragma unroll
    for (int b = 0; b < 4; ++b) red[ty * kSimtKeys + tx + 16 * b] = col[b];
    __syncthreads();
    if (threadIdx.x < kSimtKeys && j0 + threadIdx.x < N) {
        float s = 0.f;
#pragma unroll
        for (int t = 0; t < 16; ++t) s += red[t * kSimtKeys + threadIdx.x];
        scores[(size_t)unit * N + j0 + threadIdx.x] = s;
    }
}

}  // namespace ipotk
