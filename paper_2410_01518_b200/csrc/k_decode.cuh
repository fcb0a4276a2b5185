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

// The end of a block's work: dec_sm holds, per warp and head, the unnormalised output (d floats), the reference
// exponent and the sum.  The warps are merged into the block's entry of `partial`; the block that finishes a unit
// last merges the unit's splits and writes the normalised output and the log-sum-exp.
__device__ __forceinline__ void dec_finish(const float *dec_sm, int warps, int G, int d, int unit, int split, int splits,
                                           float *partial, int *counters, float *__restrict__ out, float *__restrict__ lse, int *is_last)
{
    const int ds = d + 2;
    __syncthreads();
    float *dst = partial + ((size_t)unit * splits + split) * G * ds;
    for (int e = threadIdx.x; e < G * ds; e += blockDim.x) {
        const int h = e / ds, c = e - h * ds;
        float ref = -INFINITY;
        for (int w = 0; w < warps; ++w) ref = fmaxf(ref, dec_sm[((size_t)w * G + h) * ds + d]);
        float v;
        if (c == d) {
            v = ref;
        } else {
            v = 0.f;
            for (int w = 0; w < warps; ++w) {
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
        *is_last = done == splits - 1;
        if (*is_last && splits > 1) counters[unit] = 0;  // ready for the next call
    }
    __syncthreads();
    if (!*is_last) return;
    __threadfence();
    const float *src = partial + (size_t)unit * splits * G * ds;
    for (int e = threadIdx.x; e < G * d; e += blockDim.x) {
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
    dec_finish(dec_sm, kDecWarps, G, d, unit, split, splits, partial, counters, out, lse, &is_last);
}


// ------------------------------------------------------------------ bf16 pots: the same stream on warp-level tensor cores
// The fp32 path above spends ~50 instructions per key on unpacking, FMAs and shuffle sums, which keeps it at 0.6
// of the HBM roofline.  For bf16 rows both products are m16n8k16 tiles with fp32 accumulation: S^T = q K^T with the
// G (<= 8) query heads padded to 16 rows, and O += P V with the weights split into two bf16 terms (p = hi + lo,
// 16 mantissa bits), so nothing is rounded to bf16 precision.  tcgen05 does not fit: its smallest tile has 64 rows
// and its accumulator layout puts keys across TMEM lanes, where the softmax would need cross-lane work.
// A warp owns 16-key tiles and its own ring of cp.async stages (keys and values, 16-byte vectors XOR-swizzled by
// row so that ldmatrix reads without bank conflicts); only __syncwarp orders the ring.
constexpr int kMmaWarps = 4;
constexpr int kMmaStages = 3;

__host__ __device__ inline size_t decode_mma_smem_bytes(int G, int d)
{
    const size_t ring = (size_t)kMmaWarps * kMmaStages * 2 * 16 * d * 2, merge = (size_t)kMmaWarps * G * (d + 2) * sizeof(float);
    return ring > merge ? ring : merge;
}

__device__ __forceinline__ void dec_cp_async16_zfill(void *smem_dst, const void *gmem_src, bool valid)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src),
                 "r"(valid ? 16 : 0) : "memory");
}
__device__ __forceinline__ void dec_ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void dec_ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void dec_mma(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t dec_pack_bf16(float lo, float hi)
{
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h);
}

// grid (splits, units), block 128.  D = head dimension (64 or 128), G <= 8 at run time.
template <int D>
__global__ void __launch_bounds__(kMmaWarps * 32)
decode_attn_mma_kernel(const __nv_bfloat16 *__restrict__ Kp, const __nv_bfloat16 *__restrict__ Vp, const __nv_bfloat16 *__restrict__ q,
                       float *__restrict__ out, float *__restrict__ lse, float *partial, int *counters, int N, int G,
                       size_t unit_elems, float scale_log2e)
{
    constexpr int VPR = D / 8;          // 16-byte vectors per row
    constexpr int NT = D / 8;           // output column tiles of 8
    constexpr int STAGE_VECS = 16 * VPR;  // vectors of keys (and of values) per stage
    extern __shared__ __align__(16) uint8_t dec_raw[];
    __shared__ int is_last;
    const int unit = blockIdx.y, split = blockIdx.x, splits = gridDim.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, quad = lane >> 2, tq = lane & 3;
    const int per = (N + splits - 1) / splits, k0 = split * per, k1 = min(N, k0 + per);
    const int tiles = k1 > k0 ? (k1 - k0 + 15) / 16 : 0;
    const int my_tiles = tiles > warp ? (tiles - warp + kMmaWarps - 1) / kMmaWarps : 0;  // tiles warp, warp + 4, ...
    const uint4 *Kg = reinterpret_cast<const uint4 *>(Kp + (size_t)unit * unit_elems);
    const uint4 *Vg = reinterpret_cast<const uint4 *>(Vp + (size_t)unit * unit_elems);
    uint4 *ring = reinterpret_cast<uint4 *>(dec_raw) + (size_t)warp * kMmaStages * 2 * STAGE_VECS;

    auto issue = [&](int i) {  // this warp's i-th tile into stage i % kMmaStages
        if (i < my_tiles) {
            const int key0 = k0 + (warp + i * kMmaWarps) * 16;
            uint4 *sk = ring + (size_t)(i % kMmaStages) * 2 * STAGE_VECS, *sv = sk + STAGE_VECS;
#pragma unroll
            for (int u = 0; u < STAGE_VECS / 32; ++u) {
                const int v = u * 32 + lane, r = v / VPR, c = v - r * VPR;
                const bool ok = key0 + r < k1;
                const size_t g = (size_t)(ok ? key0 + r : k0) * VPR + c;
                const int dsti = r * VPR + (c ^ (r & 7));
                dec_cp_async16_zfill(sk + dsti, Kg + g, ok);  // rows beyond the range become zeros
                dec_cp_async16_zfill(sv + dsti, Vg + g, ok);
            }
        }
        dec_cp_async_commit();
    };

    // A fragments of the queries: rows = heads (quad), rows >= G and rows 8..15 are zero
    uint32_t qa[D / 16][2];
    {
        const uint32_t *qr = reinterpret_cast<const uint32_t *>(q + ((size_t)unit * G + min(quad, G - 1)) * D);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            qa[ks][0] = quad < G ? __ldg(qr + ks * 8 + tq) : 0u;
            qa[ks][1] = quad < G ? __ldg(qr + ks * 8 + 4 + tq) : 0u;
        }
    }
    float o[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
    float m = -INFINITY, l = 0.f;  // of head `quad`; l is this lane's share of the sum

#pragma unroll
    for (int i = 0; i < kMmaStages - 1; ++i) issue(i);
    for (int i = 0; i < my_tiles; ++i) {
        dec_cp_async_wait<kMmaStages - 2>();
        __syncwarp();  // every lane's copies of tile i are in; every lane is done with the stage refilled next
        issue(i + kMmaStages - 1);
        const uint32_t sk = (uint32_t)__cvta_generic_to_shared(ring + (size_t)(i % kMmaStages) * 2 * STAGE_VECS);
        const uint32_t sv = sk + STAGE_VECS * 16;
        const int key0 = k0 + (warp + i * kMmaWarps) * 16;
        // ---- S^T = q K^T for 16 keys: two column tiles of 8 keys
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
        {
            const int r = (lane & 7) + ((lane >> 4) & 1) * 8, cs = (lane >> 3) & 1;  // row and low/high 8 channels this lane addresses
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                uint32_t b[4];
                dec_ldmatrix_x4(b, sk + (uint32_t)(r * VPR + ((2 * ks + cs) ^ (r & 7))) * 16);
                dec_mma(s0, qa[ks][0], 0u, qa[ks][1], 0u, b[0], b[1]);
                dec_mma(s1, qa[ks][0], 0u, qa[ks][1], 0u, b[2], b[3]);
            }
        }
        // this lane: head `quad`, keys key0 + 2 tq, + 1 (s0[0], s0[1]) and key0 + 8 + 2 tq, + 1 (s1[0], s1[1])
        float sc[4] = {s0[0] * scale_log2e, s0[1] * scale_log2e, s1[0] * scale_log2e, s1[1] * scale_log2e};
        const int kk[4] = {key0 + 2 * tq, key0 + 2 * tq + 1, key0 + 8 + 2 * tq, key0 + 9 + 2 * tq};
        float mt = -INFINITY;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (kk[j] >= k1) sc[j] = -INFINITY;
            mt = fmaxf(mt, sc[j]);
        }
        mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 1));
        mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 2));
        const float mn = fmaxf(m, mt);  // tile 0 always has a valid key, so mn is finite
        if (__any_sync(0xffffffffu, mn > m)) {
            const float corr = dec_scale(m, mn);
            l *= corr;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                o[nt][0] *= corr;
                o[nt][1] *= corr;
            }
            m = mn;
        }
        float p[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            p[j] = dec_ex2(sc[j] - m);  // -inf -> 0
            l += p[j];
        }
        // weights as two bf16 terms; A fragments of P (rows = heads, columns = the tile's 16 keys)
        float ph[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) ph[j] = __bfloat162float(__float2bfloat16_rn(p[j]));
        const uint32_t ah0 = dec_pack_bf16(ph[0], ph[1]), ah2 = dec_pack_bf16(ph[2], ph[3]);
        const uint32_t al0 = dec_pack_bf16(p[0] - ph[0], p[1] - ph[1]), al2 = dec_pack_bf16(p[2] - ph[2], p[3] - ph[3]);
        // ---- O += P V, two output column tiles per ldmatrix
        {
            const int r = (lane & 7) + ((lane >> 3) & 1) * 8, cv = lane >> 4;
#pragma unroll
            for (int nt = 0; nt < NT; nt += 2) {
                uint32_t b[4];
                dec_ldmatrix_x4_trans(b, sv + (uint32_t)(r * VPR + ((nt + cv) ^ (r & 7))) * 16);
                dec_mma(o[nt], ah0, 0u, ah2, 0u, b[0], b[1]);
                dec_mma(o[nt], al0, 0u, al2, 0u, b[0], b[1]);
                dec_mma(o[nt + 1], ah0, 0u, ah2, 0u, b[2], b[3]);
                dec_mma(o[nt + 1], al0, 0u, al2, 0u, b[2], b[3]);
            }
        }
    }
    dec_cp_async_wait<0>();
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    __syncthreads();  // every warp has left its ring: the memory now carries the merge of the warps
    float *dec_sm = reinterpret_cast<float *>(dec_raw);
    const int ds = D + 2;
    if (quad < G) {
        float *row = dec_sm + ((size_t)warp * G + quad) * ds;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            row[nt * 8 + 2 * tq] = o[nt][0];
            row[nt * 8 + 2 * tq + 1] = o[nt][1];
        }
        if (tq == 0) {
            row[D] = m;
            row[D + 1] = l;
        }
    }
    dec_finish(dec_sm, kMmaWarps, G, D, unit, split, splits, partial, counters, out, lse, &is_last);
}

}  // namespace ipotk
