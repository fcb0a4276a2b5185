// Row movers of the pot:
//   append_kernel  : Sec. 3.2 - new rows go into the free slots behind the survivors, in order;
//   compact_kernel : Appendix B "KV-cache compression" - K'[r] = K[idx[r]],
//                    V'[r] = V[idx[r]] - done in place.
// Both move 16-byte vectors.
#pragma once
#include "common.cuh"

namespace ipotk {

constexpr int kMoveThreads = 256;
constexpr int kMoveVecs = 8;  // 16-byte vectors in flight per thread

// One block's share of a copy of n_vecs vectors: pieces blocks of kMoveThreads threads, block `piece`.
__device__ __forceinline__ void append_body(const uint4 *__restrict__ src, uint4 *__restrict__ dst, size_t n_vecs, int piece, int pieces)
{
    const size_t stride = (size_t)pieces * kMoveThreads;
    size_t v = (size_t)piece * kMoveThreads + threadIdx.x;
    for (; v + (kMoveVecs - 1) * stride < n_vecs; v += kMoveVecs * stride) {
        uint4 t[kMoveVecs];
#pragma unroll
        for (int i = 0; i < kMoveVecs; ++i) t[i] = __ldg(src + v + i * stride);
#pragma unroll
        for (int i = 0; i < kMoveVecs; ++i) dst[v + i * stride] = t[i];
    }
    for (; v < n_vecs; v += stride) dst[v] = __ldg(src + v);
}

// grid (pieces, units, 1 or 2): tensor z of unit y (z = 0 alone: the first pair of pointers); src is [units][n_vecs],
// dst is the pot.
__global__ void __launch_bounds__(kMoveThreads)
append_kernel(const uint4 *__restrict__ srcK, const uint4 *__restrict__ srcV, uint4 *__restrict__ potK,
              uint4 *__restrict__ potV, size_t n_vecs, size_t unit_vecs, size_t first_vec)
{
    const uint4 *src = (blockIdx.z ? srcV : srcK) + (size_t)blockIdx.y * n_vecs;
    uint4 *dst = (blockIdx.z ? potV : potK) + (size_t)blockIdx.y * unit_vecs + first_vec;
    append_body(src, dst, n_vecs, blockIdx.x, gridDim.x);
}

// In-place gather.  grid (slices, 2, units).  A block owns byte columns
// [slice * slice_vecs, (slice + 1) * slice_vecs) (in 16-byte vectors) of every
// row of one tensor of one unit, so blocks never touch the same bytes.  idx is
// ascending, hence idx[r] >= r: the block walks the rows in ascending chunks,
// reads a whole chunk into registers, synchronises, then writes it.  A chunk's
// writes land in rows below the next chunk's first row, and every later source
// row lies at or above it, so nothing that is still needed is overwritten.
// Rows with idx[r] == r are left alone.
// base: the block's first vector of row 0 (its byte-column slice of one tensor of one unit).
// Rows from alt_first on may still lie outside the pot, in the caller's chunk of a deferred append: alt is then the
// block's first vector of the chunk's row 0 (same byte columns; slot alt_first), else alt_first = INT_MAX.  Such
// rows are fetched from there, also when they keep their slot number, so after the gather the pot holds every
// survivor and nothing else of the chunk was ever copied.
__device__ __forceinline__ void compact_body(uint4 *__restrict__ base, const int32_t *__restrict__ ix, int keep, int N,
                                             int row_vecs, int slice_vecs, int *status, const uint4 *__restrict__ alt = nullptr,
                                             int alt_first = 0x7fffffff)
{
    const int rows_per_pass = kMoveThreads / slice_vecs;  // rows covered by one vector per thread
    const int chunk_rows = rows_per_pass * kMoveVecs;
    const int my_row = threadIdx.x / slice_vecs, my_vec = threadIdx.x - my_row * slice_vecs;
    for (int r0 = 0; r0 < keep; r0 += chunk_rows) {
        uint4 t[kMoveVecs];
        int src[kMoveVecs];
#pragma unroll
        for (int i = 0; i < kMoveVecs; ++i) {
            const int r = r0 + i * rows_per_pass + my_row;
            src[i] = -1;
            if (r < keep && my_row < rows_per_pass) {
                const int s = ix[r];
                if (s < r || s >= N) set_status(status, kStatusBounds);
                else if (s != r || s >= alt_first) src[i] = s;
            }
        }
#pragma unroll
        for (int i = 0; i < kMoveVecs; ++i)
            if (src[i] >= 0)
                t[i] = src[i] >= alt_first ? __ldg(alt + (size_t)(src[i] - alt_first) * row_vecs + my_vec)
                                           : base[(size_t)src[i] * row_vecs + my_vec];
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kMoveVecs; ++i) {
            const int r = r0 + i * rows_per_pass + my_row;
            if (src[i] >= 0) base[(size_t)r * row_vecs + my_vec] = t[i];
        }
    }
}

// A deferred append's chunk: rows of slot numbers first, first + 1, ... of every unit, still in the caller's buffers
// ([units][rows][row_vecs]); K or V is NULL where the pot already holds those rows.
struct PendingRows {
    const uint4 *K, *V;
    size_t unit_vecs;  // rows * row_vecs
    int first;
};

__global__ void __launch_bounds__(kMoveThreads)
compact_kernel(uint4 *__restrict__ potK, uint4 *__restrict__ potV, const int32_t *__restrict__ idx,
               int keep, int N, int row_vecs, int slice_vecs, size_t unit_vecs, int *status, PendingRows pend)
{
    // Block order: the units from the last one down, K then V of a unit next to each other.  The scorer of the next
    // cycle starts at unit 0 and finds the rows written last still in L2, and the two tensors of a unit share their
    // index list while it is hot (measured against units ascending, all K before all V: step 183.2 -> 181.3 us).
    const unsigned unit = gridDim.z - 1 - blockIdx.z, tensor = blockIdx.y;
    uint4 *base = (tensor ? potV : potK) + (size_t)unit * unit_vecs + (size_t)blockIdx.x * slice_vecs;
    // launched as a programmatic dependent of the selection: the blocks may be resident before it has ended and
    // wait here for its index lists (returns at once after an ordinary launch)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint4 *alt = tensor ? pend.V : pend.K;
    if (alt) alt += (size_t)unit * pend.unit_vecs + (size_t)blockIdx.x * slice_vecs;
    compact_body(base, idx + (size_t)unit * keep, keep, N, row_vecs, slice_vecs, status, alt, alt ? pend.first : 0x7fffffff);
}

}  // namespace ipotk
