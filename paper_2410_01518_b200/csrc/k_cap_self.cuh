// The CaP's own keys inside the softmax (Appendix B, "Calculate Attention Score": the CaP queries attend to
// every key of the sequence under the causal mask, the CaP columns are cut away afterwards).  For query row r
// (CaP position i = r % P of one of the G query heads) this kernel produces (max, sum 2^(x - max)) over the
// CaP keys 0..i in log2 units; the scorers merge the pair into the row's denominator.
//
// The work is tiny (M x P x d per unit), so it runs beside the main scorer as one small launch: bf16 rows with
// d a multiple of 16 go through warp-level m16n8k16 tensor-core tiles (a block stages 64 query rows and up to
// 64 CaP keys in padded shared memory, a warp owns 16 rows); everything else uses the generic row-statistics
// kernel of the fp32 scorer with a causal limit.
#pragma once
#include <cuda_bf16.h>

#include "common.cuh"

namespace ipotk {

constexpr int kSelfWarps = 4;        // warps per block, 16 query rows each
constexpr int kSelfRows = kSelfWarps * 16;
constexpr int kSelfKeys = 64;        // CaP keys staged per pass
constexpr int kSelfPad = 8;          // bf16 elements of padding per staged row: fragment reads hit 32 different banks

__host__ __device__ inline size_t self_smem_bytes(int d) { return (size_t)(kSelfRows + kSelfKeys) * (d + kSelfPad) * 2; }

__device__ __forceinline__ void mma_bf16_16x8x16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void self_merge(float &m, float &l, float m2, float l2)
{
    const float mn = fmaxf(m, m2);
    const float a = (m == -INFINITY) ? 0.f : l * exp2f(m - mn);
    const float b = (m2 == -INFINITY) ? 0.f : l2 * exp2f(m2 - mn);
    m = mn;
    l = a + b;
}

// Rows [row0, row0 + n) of a [limit][d] bf16 matrix -> shared memory, row stride d + kSelfPad, with 16-byte
// loads; rows at or beyond `limit` repeat the last row (their results are masked or not stored).
__device__ __forceinline__ void self_stage(__nv_bfloat16 *dst, const __nv_bfloat16 *src, int row0, int n, int limit, int d)
{
    const int vpr = d / 8, ds = d + kSelfPad;
    for (int v = threadIdx.x; v < n * vpr; v += kSelfWarps * 32) {
        const int r = v / vpr, c = (v - r * vpr) * 8;
        *reinterpret_cast<uint4 *>(dst + r * ds + c) =
            *reinterpret_cast<const uint4 *>(src + (size_t)min(row0 + r, limit - 1) * d + c);
    }
}

// grid (ceil(M / 64), units), block 128, dynamic shared memory self_smem_bytes(d).
// Q [units][M][d], Kc [units][P][d] bf16, d a multiple of 16; out [units][M] (max, sum).
__global__ void __launch_bounds__(kSelfWarps * 32)
cap_self_stats_bf16(const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ Kc, float2 *__restrict__ out,
                    int M, int P, int d, float scale_log2e)
{
    extern __shared__ __align__(16) uint8_t self_sm[];
    __nv_bfloat16 *Qs = reinterpret_cast<__nv_bfloat16 *>(self_sm);
    __nv_bfloat16 *Ks = Qs + kSelfRows * (d + kSelfPad);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int unit = blockIdx.y, brow0 = blockIdx.x * kSelfRows;
    const int ksteps = d / 16, ws = (d + kSelfPad) / 2;  // row stride in 32-bit words
    const int r[2] = {brow0 + warp * 16 + g, brow0 + warp * 16 + g + 8};
    const int lim[2] = {r[0] % P + 1, r[1] % P + 1};  // CaP keys each row may see
    // the largest limit among the block's 64 consecutive rows: P if they wrap around a head boundary
    const int first = brow0 % P;
    const int block_lim = (first + kSelfRows - 1 >= P) ? P : first + kSelfRows;
    self_stage(Qs, Q + (size_t)unit * M * d, brow0, kSelfRows, M, d);
    float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
    const uint32_t *qa = reinterpret_cast<const uint32_t *>(Qs) + (warp * 16 + g) * ws;
    for (int kb = 0; kb < block_lim; kb += kSelfKeys) {
        if (kb > 0) __syncthreads();  // the previous pass has read Ks
        self_stage(Ks, Kc + (size_t)unit * P * d, kb, kSelfKeys, P, d);  // the first pass loads beside the query rows
        __syncthreads();
        const int tiles = min(kSelfKeys, block_lim - kb);
        for (int n0 = 0; n0 < tiles; n0 += 8) {
            const uint32_t *kr = reinterpret_cast<const uint32_t *>(Ks) + (n0 + g) * ws;
            float c[4] = {0.f, 0.f, 0.f, 0.f};
            for (int ks = 0; ks < ksteps; ++ks) {
                const uint32_t a[4] = {qa[ks * 8 + t], qa[8 * ws + ks * 8 + t], qa[ks * 8 + 4 + t], qa[8 * ws + ks * 8 + 4 + t]};
                mma_bf16_16x8x16(c, a, kr[ks * 8 + t], kr[ks * 8 + 4 + t]);
            }
            // c[0], c[1]: row r[0], keys kb + n0 + 2t, + 1;  c[2], c[3]: row r[1], same keys
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const float x0 = c[2 * h] * scale_log2e, x1 = c[2 * h + 1] * scale_log2e;
                const int key = kb + n0 + 2 * t;
                const bool v0 = key < lim[h], v1 = key + 1 < lim[h];
                const float tm = fmaxf(v0 ? x0 : -INFINITY, v1 ? x1 : -INFINITY);
                if (tm > -INFINITY) self_merge(m[h], l[h], tm, (v0 ? exp2f(x0 - tm) : 0.f) + (v1 ? exp2f(x1 - tm) : 0.f));
            }
        }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
#pragma unroll
        for (int off = 1; off <= 2; off <<= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, m[h], off);
            const float l2 = __shfl_xor_sync(0xffffffffu, l[h], off);
            self_merge(m[h], l[h], m2, l2);
        }
        if (t == 0 && r[h] < M) out[(size_t)unit * M + r[h]] = make_float2(m[h], l[h]);
    }
}

}  // namespace ipotk
