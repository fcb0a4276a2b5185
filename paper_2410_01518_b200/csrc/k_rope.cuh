// Context-reset rotary embedding (Sec. 3.4) fused into the row movers.  The pot keeps its keys without rotary
// embedding; beside it lives a rotated copy in which slot j carries position j, the copy the CaP queries (and the
// model's attention) read.  Positions only change when rows move, so the two kernels that move rows also write
// the rotated copy:
//   append_rope_kernel  : new key rows -> pot rows [first_row, first_row + n) unrotated, and rotated at those
//                         positions into the copy;
//   compact_rope_kernel : the in-place gather of compact_kernel on the unrotated keys; every moved row is also
//                         rotated at its new slot number into the copy.  Rows that stay where they are keep
//                         their rotated row.
// Both are HBM-bound copies with idle ALUs, so the rotation costs its extra store traffic only, and no separate
// pass over the pot follows a cycle.
//
// The rotation (the paper gives no detail; tables are the caller's, in the pot's storage type): channel pairs
// (c, c + d/2) or (2c, 2c + 1), frequency index c, single precision, exactly
//   lo' = fma(lo, cos, -(hi * sin)),  hi' = fma(hi, cos, lo * sin),  rounded once to the storage type.
// A thread handles two 16-byte vectors of a row, vector g and vector g + row_vecs / 2: for the half pairing
// they are each other's partners, for the interleaved pairing each holds whole pairs.
#pragma once
#include "common.cuh"
#include "k_move.cuh"

namespace ipotk {

constexpr int kRopeVecs = 4;  // row pairs of vectors in flight per thread in compact_rope_kernel

template <typename T> struct RopeVec;
template <> struct RopeVec<float> {
    static constexpr int kElems = 4;
    __device__ static __forceinline__ void unpack(const uint4 &v, float *x)
    {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y); x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    }
    __device__ static __forceinline__ uint4 pack(const float *x)
    {
        return make_uint4(__float_as_uint(x[0]), __float_as_uint(x[1]), __float_as_uint(x[2]), __float_as_uint(x[3]));
    }
};
template <> struct RopeVec<__nv_bfloat16> {
    static constexpr int kElems = 8;
    __device__ static __forceinline__ void unpack(const uint4 &v, float *x)
    {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    __device__ static __forceinline__ uint4 pack(const float *x)
    {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);  // nearest even
            w[i] = *reinterpret_cast<const uint32_t *>(&h);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};

__device__ __forceinline__ void rope_pair(float lo, float hi, float cs, float sn, float &lo_out, float &hi_out)
{
    lo_out = __fmaf_rn(lo, cs, -__fmul_rn(hi, sn));
    hi_out = __fmaf_rn(hi, cs, __fmul_rn(lo, sn));
}

// The table vectors a thread needs for vectors g and g + half_vecs of a row at position pos (cos_t, sin_t:
// [positions][d / 2]): half pairing - cos and sin of frequencies g * VE .. (2 vectors); interleaved - a vector
// holds VE / 2 pairs, so each of the two data vectors needs half a table vector, fetched as the 16-byte vector
// that contains it (4 vectors: cos a, sin a, cos b, sin b).
template <typename T, bool kInterleaved> struct RopeTab {
    uint4 v[kInterleaved ? 4 : 2];
    __device__ __forceinline__ void load(int g, int half_vecs, int pos, const T *__restrict__ cos_t, const T *__restrict__ sin_t)
    {
        constexpr int VE = RopeVec<T>::kElems;
        const size_t trow = (size_t)pos * half_vecs * VE;  // d / 2 = half_vecs * VE table entries per position
        if (!kInterleaved) {
            v[0] = __ldg(reinterpret_cast<const uint4 *>(cos_t + trow + (size_t)g * VE));
            v[1] = __ldg(reinterpret_cast<const uint4 *>(sin_t + trow + (size_t)g * VE));
        } else {
            const int fa = g * (VE / 2), fb = (g + half_vecs) * (VE / 2);
            v[0] = __ldg(reinterpret_cast<const uint4 *>(cos_t + trow + (fa / VE) * VE));
            v[1] = __ldg(reinterpret_cast<const uint4 *>(sin_t + trow + (fa / VE) * VE));
            v[2] = __ldg(reinterpret_cast<const uint4 *>(cos_t + trow + (fb / VE) * VE));
            v[3] = __ldg(reinterpret_cast<const uint4 *>(sin_t + trow + (fb / VE) * VE));
        }
    }
};

// Rotates vectors g (a) and g + half_vecs (b) of a row with the table vectors loaded for its position.
template <typename T, bool kInterleaved>
__device__ __forceinline__ void rope_apply(const uint4 &a, const uint4 &b, int g, int half_vecs, const RopeTab<T, kInterleaved> &tab,
                                           uint4 &a_out, uint4 &b_out)
{
    constexpr int VE = RopeVec<T>::kElems;
    float xa[VE], xb[VE], ya[VE], yb[VE];
    RopeVec<T>::unpack(a, xa);
    RopeVec<T>::unpack(b, xb);
    if (!kInterleaved) {
        // a holds channels g * VE .. (the "lo" halves), b their partners c + d/2; frequencies g * VE ..
        float cs[VE], sn[VE];
        RopeVec<T>::unpack(tab.v[0], cs);
        RopeVec<T>::unpack(tab.v[1], sn);
#pragma unroll
        for (int i = 0; i < VE; ++i) rope_pair(xa[i], xb[i], cs[i], sn[i], ya[i], yb[i]);
    } else {
        // vector v holds the pairs (2c, 2c + 1) with c = v * VE / 2 ..
        float csa[VE], sna[VE], csb[VE], snb[VE];
        RopeVec<T>::unpack(tab.v[0], csa);
        RopeVec<T>::unpack(tab.v[1], sna);
        RopeVec<T>::unpack(tab.v[kInterleaved ? 2 : 0], csb);
        RopeVec<T>::unpack(tab.v[kInterleaved ? 3 : 1], snb);
        const int oa = (g * (VE / 2)) % VE, ob = ((g + half_vecs) * (VE / 2)) % VE;  // 0 or VE / 2
#pragma unroll
        for (int i = 0; i < VE / 2; ++i) {
            rope_pair(xa[2 * i], xa[2 * i + 1], oa ? csa[VE / 2 + i] : csa[i], oa ? sna[VE / 2 + i] : sna[i], ya[2 * i], ya[2 * i + 1]);
            rope_pair(xb[2 * i], xb[2 * i + 1], ob ? csb[VE / 2 + i] : csb[i], ob ? snb[VE / 2 + i] : snb[i], yb[2 * i], yb[2 * i + 1]);
        }
    }
    a_out = RopeVec<T>::pack(ya);
    b_out = RopeVec<T>::pack(yb);
}

template <typename T, bool kInterleaved>
__device__ __forceinline__ void rope_two_vectors(const uint4 &a, const uint4 &b, int g, int half_vecs, int pos,
                                                 const T *__restrict__ cos_t, const T *__restrict__ sin_t,
                                                 uint4 &a_out, uint4 &b_out)
{
    RopeTab<T, kInterleaved> tab;
    tab.load(g, half_vecs, pos, cos_t, sin_t);
    rope_apply<T, kInterleaved>(a, b, g, half_vecs, tab, a_out, b_out);
}

// grid (pieces, units, 2 or 1).  z = 0: src: key rows of unit y at src + y * src_unit_vecs, n rows of row_vecs vectors;
// the rows go to pot rows first_row ... of potK (unchanged) and potKrot (rotated at their slot numbers).  src may be
// the pot rows themselves (rows that a host copy already put in place): the plain copy then rewrites them as they
// are.  z = 1: the value rows, a plain copy as in append_kernel (srcV is [units][n * row_vecs]).
template <typename T, bool kInterleaved>
__global__ void __launch_bounds__(kMoveThreads)
append_rope_kernel(const uint4 *__restrict__ src, size_t src_unit_vecs, uint4 *potK, uint4 *__restrict__ potKrot,
                   const T *__restrict__ cos_t, const T *__restrict__ sin_t, int n, int row_vecs, size_t unit_vecs, int first_row,
                   const uint4 *__restrict__ srcV, uint4 *__restrict__ potV)
{
    if (blockIdx.z == 1) {
        const size_t n_vecs = (size_t)n * row_vecs;
        append_body(srcV + (size_t)blockIdx.y * n_vecs, potV + (size_t)blockIdx.y * unit_vecs + (size_t)first_row * row_vecs,
                    n_vecs, blockIdx.x, gridDim.x);
        return;
    }
    const int half_vecs = row_vecs / 2;
    const uint4 *s = src + (size_t)blockIdx.y * src_unit_vecs;
    uint4 *dk = potK + (size_t)blockIdx.y * unit_vecs + (size_t)first_row * row_vecs;
    uint4 *dr = potKrot + (size_t)blockIdx.y * unit_vecs + (size_t)first_row * row_vecs;
    const size_t items = (size_t)n * half_vecs, stride = (size_t)gridDim.x * kMoveThreads;
    size_t it = (size_t)blockIdx.x * kMoveThreads + threadIdx.x;
    for (; it + stride < items; it += 2 * stride) {  // two items (four loads) in flight
        size_t ia[2], ib[2];
        int g[2], r[2];
        uint4 a[2], b[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const size_t item = it + u * stride;
            r[u] = (int)(item / half_vecs);
            g[u] = (int)(item - (size_t)r[u] * half_vecs);
            ia[u] = (size_t)r[u] * row_vecs + g[u];
            ib[u] = ia[u] + half_vecs;
            a[u] = s[ia[u]];
            b[u] = s[ib[u]];
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            uint4 ra, rb;
            rope_two_vectors<T, kInterleaved>(a[u], b[u], g[u], half_vecs, first_row + r[u], cos_t, sin_t, ra, rb);
            dk[ia[u]] = a[u];
            dk[ib[u]] = b[u];
            dr[ia[u]] = ra;
            dr[ib[u]] = rb;
        }
    }
    for (; it < items; it += stride) {
        const int r = (int)(it / half_vecs), g = (int)(it - (size_t)r * half_vecs);
        const size_t ia = (size_t)r * row_vecs + g, ib = ia + half_vecs;
        const uint4 a = s[ia], b = s[ib];
        uint4 ra, rb;
        rope_two_vectors<T, kInterleaved>(a, b, g, half_vecs, first_row + r, cos_t, sin_t, ra, rb);
        dk[ia] = a;
        dk[ib] = b;
        dr[ia] = ra;
        dr[ib] = rb;
    }
}

// In-place gather of the unrotated keys with the rotated copy written beside it.
// grid (max(k_slices, v_slices), units, 2).  For z = 0 a block
// owns the vector pairs (g, g + row_vecs / 2) with g in [slice * slice_vecs, (slice + 1) * slice_vecs) of every row
// of one unit; the walk over the rows is compact_kernel's (ascending chunks, read - barrier - write), which is
// safe in place because idx[r] >= r.  The rotated copy is only written, never read.
// z = 1 (if launched): the value rows, compact_kernel's walk with its own slicing (v_slices slices of v_slice_vecs);
// pend.V names the value rows of a deferred append, if any (pend.K is not used: the keys are in the pot).
template <typename T, bool kInterleaved>
__global__ void __launch_bounds__(kMoveThreads)
compact_rope_kernel(uint4 *potK, uint4 *__restrict__ potKrot, const T *__restrict__ cos_t, const T *__restrict__ sin_t,
                    const int32_t *__restrict__ idx, int keep, int N, int row_vecs, int k_slices, int slice_vecs, size_t unit_vecs,
                    int *status, uint4 *potV, int v_slices, int v_slice_vecs, PendingRows pend)
{
    if (blockIdx.z == 1) {
        if ((int)blockIdx.x < v_slices) {
            const uint4 *alt = pend.V ? pend.V + (size_t)blockIdx.y * pend.unit_vecs + (size_t)blockIdx.x * v_slice_vecs : nullptr;
            compact_body(potV + (size_t)blockIdx.y * unit_vecs + (size_t)blockIdx.x * v_slice_vecs, idx + (size_t)blockIdx.y * keep,
                         keep, N, row_vecs, v_slice_vecs, status, alt, alt ? pend.first : 0x7fffffff);
        }
        return;
    }
    if ((int)blockIdx.x >= k_slices) return;
    const int half_vecs = row_vecs / 2;
    uint4 *base = potK + (size_t)blockIdx.y * unit_vecs;
    uint4 *rbase = potKrot + (size_t)blockIdx.y * unit_vecs;
    const int32_t *ix = idx + (size_t)blockIdx.y * keep;
    const int rows_per_pass = kMoveThreads / slice_vecs;
    const int chunk_rows = rows_per_pass * kRopeVecs;
    const int my_row = threadIdx.x / slice_vecs, g = blockIdx.x * slice_vecs + (threadIdx.x - my_row * slice_vecs);
    for (int r0 = 0; r0 < keep; r0 += chunk_rows) {
        uint4 ta[kRopeVecs], tb[kRopeVecs];
        int src[kRopeVecs];
#pragma unroll
        for (int i = 0; i < kRopeVecs; ++i) {
            const int r = r0 + i * rows_per_pass + my_row;
            src[i] = -1;
            if (r < keep && my_row < rows_per_pass) {
                const int s = ix[r];
                if (s < r || s >= N) set_status(status, kStatusBounds);
                else if (s != r) src[i] = s;
            }
        }
#pragma unroll
        for (int i = 0; i < kRopeVecs; ++i) {
            if (src[i] >= 0) {
                ta[i] = base[(size_t)src[i] * row_vecs + g];
                tb[i] = base[(size_t)src[i] * row_vecs + g + half_vecs];
            }
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kRopeVecs; ++i) {
            const int r = r0 + i * rows_per_pass + my_row;
            if (src[i] >= 0) {
                uint4 ra, rb;
                // the table vectors are fetched here, not with the rows: holding them across the barrier costs a
                // third of the resident blocks (measured: 164 us against 142 us on the 32-layer workload)
                rope_two_vectors<T, kInterleaved>(ta[i], tb[i], g, half_vecs, r, cos_t, sin_t, ra, rb);
                base[(size_t)r * row_vecs + g] = ta[i];
                base[(size_t)r * row_vecs + g + half_vecs] = tb[i];
                rbase[(size_t)r * row_vecs + g] = ra;
                rbase[(size_t)r * row_vecs + g + half_vecs] = rb;
            }
        }
    }
}

}  // namespace ipotk
