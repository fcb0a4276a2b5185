// CaP scoring on the 5th-generation tensor cores (Sec. 3.3.1, Eq. 2), bf16, d = 128 or 64.
//
// Item  = (unit, block of 128 folded query rows): one row-softmax problem over the
//         unit's N pot keys.
// Task  = (item, slab of 256 keys).  Tasks are numbered item-major and dealt round
//         robin to a persistent grid of one CTA per SM, so the slabs of an item are
//         in flight on neighbouring SMs at the same time.
//
// Per task, inside one CTA (warp-specialised, two tasks in flight):
//   TMA      Q tile (128 x 128 bf16) and the slab's keys (256 x 128 bf16) land in
//            shared memory in the 128-byte-swizzled K-major layout (2 stages);
//   tcgen05  S = Q K^T (128 x 256 fp32) accumulates in one of two 256-column tensor
//            memory buffers, one 128-column half at a time: the logits never leave
//            the SM;
//   pass 1   (16 epilogue warps; a thread owns one query row x two chunks of 32 columns,
//            one in each half of the buffer) per chunk: maximum, e = 2^(x - max)
//            written back over the logits, sum - one tensor-memory read and one
//            write per logit; a quarter of the exponentials run on the FMA pipe; the chunks move
//            through two sets of 16 registers, the second chunk's first half being fetched behind the
//            exponentials of the first chunk's second half;
//   combine  (4 warps, one thread per query row) merges the eight (max, sum) pairs of
//            its row into the slab's statistics and publishes them with one 8-byte
//            store whose sum carries the launch's sign as a "fresh" mark; then reads
//            the row's statistics of all slabs of the item, re-reading until every
//            one is fresh, and turns them into the row's global maximum m, its
//            denominator l (plus, when given, the share of the CaP's own keys) and the
//            weights 2^(max_chunk - m) / l of the stored e values;
//   pass 2   (the same 16 warps, one task behind: after pass 1 of task t+1 they
//            finish task t, whose weights have arrived meanwhile)
//            u_j = sum_i e_ij 2^(max_i - m_i) / l_i as a weighted column sum: the
//            16x256b tensor-memory load shape hands every thread four rows of a
//            column pair, so the sum over a warp's 32 rows is four packed FMAs plus
//            a three-step exchange between lanes; the four warps that own the same
//            columns add their row quarters through shared memory (their own
//            128-thread barrier) and store: 256 floats per task.
// The two 128-column halves of a buffer are handed over separately (MMA -> pass 1,
// pass 2 -> MMA), so the tensor core refills one half while the other is still read.
//
// Blocks of one grid wait on each other (pass 2 needs the other slabs' statistics),
// so the grid is launched cooperatively with at most one CTA per SM: all of it is
// resident.  A CTA publishes pass 1 of task t+1 before it waits for task t, so the
// waits cannot form a cycle.  Every wait (mbarrier or statistics) is bounded by a time
// limit (a launch parameter); one that runs out records IPOT_E_TIMEOUT in the status
// word and raises a block-wide flag.  From then on every wait of the block returns at
// once: the producer and the MMA issuer stop putting work in flight and wait for what
// they have issued (loads into this CTA's shared memory, MMAs into its tensor memory)
// before the block releases tensor memory and ends; the epilogue warps run through
// their remaining iterations without waiting (their results are void).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/ipot.h"
#include "common.cuh"

namespace ipotk {

constexpr int kTcThreads = 704;      // warp 0: TMA, 1: MMA + TMEM owner, 2-17: pass 1 / pass 2, 18-21: combine
constexpr int kTcRows = 128;         // query rows per item (TMEM lanes)
constexpr int kTcSlab = 256;         // keys per task (TMEM columns per buffer)
constexpr int kTcFmaEighths = 2;     // share of pass 1's exponentials evaluated on the FMA pipe
constexpr int kTcD = 128;            // largest head dimension; 64 uses the first 64-channel half of every tile
constexpr uint32_t kTcQBytes = kTcRows * kTcD * 2;           // 32 KiB: two halves of 128 rows x 64 channels
constexpr uint32_t kTcKBytes = kTcSlab * kTcD * 2;           // 64 KiB: two halves of 256 rows x 64 channels
constexpr uint32_t kTcStageBytes = kTcQBytes + kTcKBytes;    // 96 KiB

// shared-memory carve-up (bytes from the 1024-aligned base)
constexpr uint32_t kTcOffStage = 0;                                        // [2] { Q, K }
constexpr uint32_t kTcOffColpart = 2 * kTcStageBytes;                      // [2 parities][4 row quarters][256] float
constexpr uint32_t kTcOffTstat = kTcOffColpart + 2 * 4 * kTcSlab * 4;          // [2 buffers][8 chunks][128] float2
constexpr uint32_t kTcOffFbuf = kTcOffTstat + 2 * 8 * kTcRows * 8;         // [2 buffers][8 chunks][128] float
constexpr uint32_t kTcOffBar = kTcOffFbuf + 2 * 8 * kTcRows * 4;
constexpr uint32_t kTcOffTmemSlot = kTcOffBar + 192;                       // the allocated TMEM base address
constexpr uint32_t kTcOffAbort = kTcOffBar + 196;                          // set once a wait of the CTA has run out; + 4: the block's deadline (8 bytes)
constexpr uint32_t kTcSmemBytes = kTcOffBar + 256;                         // no static shared memory: the base is 1024-aligned

// barriers: per stage Full, Empty, EReady, FReady; per (buffer, half) SFull, TEmpty at index 2 * buffer + half
enum { kBarFull = 0, kBarEmpty = 2, kBarEReady = 4, kBarFReady = 6, kBarSFull = 8, kBarTEmpty = 12, kBarDrain = 16, kBarCount = 17 };

struct TcParams {
    float *scores;        // partial array p (query rows 128p ...) at scores + p * part_stride, unit stride N
    size_t part_stride;
    float2 *stats;        // [items][slabs][128] (max in log2 units, sum * sign); all of the other sign or 0 at launch
    const float2 *cap_stats;  // NULL, or [units][M] (max, sum) over the CaP's own keys that join every row's denominator
    float sign;           // +1 or -1: this launch's "fresh" mark
    unsigned long long wait_ns;  // limit of every wait
    int withhold_cta;     // -1; test hook: this CTA never publishes its slab statistics
    int *status;
    int N, M, mtiles, slabs, tasks;
    int dhalves;          // d / 64: 64-channel halves of a tile (1 or 2)
    int new_slab0;        // slabs from this one on are read through the second key map (the chunk of a deferred
                          // append, row 0 = key 256 * new_slab0); INT_MAX if all keys are in the pot
    float scale_log2e;
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)   // never blocks
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  Every block notes a deadline (its start + the launch's wait limit) next to its give-up flag; a
// wait that is still unsatisfied then records IPOT_E_TIMEOUT and raises the flag.  Once the flag is up, later waits
// of the block return at once (false) - unless heed_flag is off, which is how a role waits for work it has itself
// put in flight before the block may end.  (Clock and flag are looked at every 1024 rounds only: the kernel's
// speed depends on this loop staying small.)
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status, bool heed_flag = true)
{
    for (uint32_t i = 0;; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 1023u) == 1023u) {
            if (heed_flag && *abort_flag) return false;
            if (global_ns() > *reinterpret_cast<volatile unsigned long long *>(abort_flag + 1)) {
                *abort_flag = 1;
                set_status(status, kStatusTimeout);
                return false;
            }
        }
    }
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 consecutive fp32 columns of this thread's TMEM lane (asynchronous: see tmem_wait_ld).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
// 16 TMEM lanes x 32 fp32 columns in the 16x256b shape: for each block j of 8 columns, thread t of the warp
// receives v[4j], v[4j+1] = lane t/4, columns 8j + 2(t%4), +1 and v[4j+2], v[4j+3] = lane t/4 + 8, same columns.
__device__ __forceinline__ void tmem_ld_16x256b_x4(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x4.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld16(uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.wait::ld.sync.aligned;"
        : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
          "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15])
        :: "memory");
}
// Waits for this thread's outstanding TMEM loads.  The loaded registers are passed
// through so that no use of them can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_wait_ld(uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.wait::ld.sync.aligned;"
        : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
          "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]),
          "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]),
          "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31])
        :: "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
        ::"r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
          "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
          "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31]),
          "r"(taddr) : "memory");
}
// 16 consecutive fp32 columns of this thread's TMEM lane (asynchronous: see tmem_wait_ld16).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};"
        ::"r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
          "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Named barrier of the four epilogue warps (one per TMEM lane quarter) that own the same columns.
// (Barrier numbers are immediates so that the kernel claims five of the SM's barriers, not all sixteen.)
__device__ __forceinline__ void column_group_sync(int cq)
{
    switch (cq) {
    case 0: asm volatile("bar.sync 1, 128;" ::: "memory"); break;
    case 1: asm volatile("bar.sync 2, 128;" ::: "memory"); break;
    case 2: asm volatile("bar.sync 3, 128;" ::: "memory"); break;
    default: asm volatile("bar.sync 4, 128;" ::: "memory"); break;
    }
}
// The slab statistics are exchanged between CTAs with single 8-byte relaxed accesses at gpu scope:
// one store publishes (max, marked sum) together, and a reader sees either the old or the new pair.
__device__ __forceinline__ float2 ld_gpu_f32x2(const float2 *p)
{
    float2 v;
    asm volatile("ld.relaxed.gpu.global.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_gpu_f32x2(float2 *p, float a, float b)
{
    asm volatile("st.relaxed.gpu.global.v2.f32 [%0], {%1, %2};" ::"l"(p), "f"(a), "f"(b) : "memory");
}
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float y;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
    return y;
}

// Maximum of 32 logits folded into four independent running maxima (no long dependency chain).
template <bool kFull>
__device__ __forceinline__ void chunk_max(const uint32_t (&v)[32], int col0, int nvalid, float (&mx)[4])
{
    if (kFull) {
#pragma unroll
        for (int i = 0; i < 32; i += 8) {
#pragma unroll
            for (int j = 0; j < 4; ++j) mx[j] = max3(mx[j], __uint_as_float(v[i + 2 * j]), __uint_as_float(v[i + 2 * j + 1]));
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (col0 + i < nvalid) mx[i & 3] = fmaxf(mx[i & 3], __uint_as_float(v[i]));
    }
}

// v <- 2^(v c - mxc) (0 beyond nvalid); the new values are also added into four packed running sums.
// kTcFmaEighths of every eight pairs are evaluated on the FMA pipe (relative error 2.7e-6, values below 2^-126
// come out as subnormal bit patterns that pass 2 multiplies like any other number): measured on the
// 256-unit 4096-key launch, 2 eighths 86.2 us, none 87.7, 3 eighths 86.8, 4 eighths 89.9.
template <bool kFull>
__device__ __forceinline__ void chunk_exp(uint32_t (&v)[32], int col0, int nvalid, float c, float mxc, float2 (&sum)[4])
{
    const float2 c2 = make_float2(c, c), nm2 = make_float2(-mxc, -mxc);
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        const float2 x = __ffma2_rn(make_float2(__uint_as_float(v[i]), __uint_as_float(v[i + 1])), c2, nm2);
        float2 e2 = pair_on_fma<kTcFmaEighths>(i >> 1) ? exp2_fma_pair(x) : make_float2(ex2(x.x), ex2(x.y));
        if (!kFull) {
            if (col0 + i >= nvalid) e2.x = 0.f;
            if (col0 + i + 1 >= nvalid) e2.y = 0.f;
        }
        sum[(i >> 1) & 3] = __fadd2_rn(sum[(i >> 1) & 3], e2);
        v[i] = __float_as_uint(e2.x);
        v[i + 1] = __float_as_uint(e2.y);
    }
}

// Pass 1 for one query row over one chunk of 32 columns (slab columns from col0): returns the chunk's
// maximum (log2 units) and the sum of e = 2^(x - max), and leaves e in tensor memory.  With no valid column
// the maximum is -inf, the sum 0 and zeros are stored.
template <bool kFull>
__device__ __forceinline__ float2 pass1_chunk(uint32_t taddr, int col0, int nvalid, float c)
{
    uint32_t v[32];
    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
    tmem_ld32(taddr, v);
    tmem_wait_ld(v);
    chunk_max<kFull>(v, col0, nvalid, mx);
    const float mxr = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
    const float mxc = (mxr == -INFINITY) ? 0.f : mxr * c;
    float2 sum[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
    chunk_exp<kFull>(v, col0, nvalid, c, mxc, sum);
    tmem_st32(taddr, v);
    const float2 s01 = __fadd2_rn(sum[0], sum[1]), s23 = __fadd2_rn(sum[2], sum[3]);
    return make_float2((mxr == -INFINITY) ? -INFINITY : mxc, (s01.x + s01.y) + (s23.x + s23.y));
}

// The same over 16 columns of a full chunk: maximum into four running maxima / exponentials into four packed sums.
// `first_pair`: index of the piece's first column pair within its chunk (it fixes which pairs take the FMA pipe).
__device__ __forceinline__ void piece_max(const uint32_t (&v)[16], float (&mx)[4])
{
#pragma unroll
    for (int i = 0; i < 16; i += 8) {
#pragma unroll
        for (int j = 0; j < 4; ++j) mx[j] = max3(mx[j], __uint_as_float(v[i + 2 * j]), __uint_as_float(v[i + 2 * j + 1]));
    }
}
template <int kFirstPair>
__device__ __forceinline__ void piece_exp(uint32_t (&v)[16], float c, float mxc, float2 (&sum)[4])
{
    const float2 c2 = make_float2(c, c), nm2 = make_float2(-mxc, -mxc);
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
        const float2 x = __ffma2_rn(make_float2(__uint_as_float(v[i]), __uint_as_float(v[i + 1])), c2, nm2);
        const float2 e2 = pair_on_fma<kTcFmaEighths>(kFirstPair + (i >> 1)) ? exp2_fma_pair(x) : make_float2(ex2(x.x), ex2(x.y));
        sum[(i >> 1) & 3] = __fadd2_rn(sum[(i >> 1) & 3], e2);
        v[i] = __float_as_uint(e2.x);
        v[i + 1] = __float_as_uint(e2.y);
    }
}
// Pass 2 for one warp over 32 rows x 32 columns: a[] and b[] are the 16x256b loads of the warp's TMEM lanes
// 0..15 and 16..31, fr2[i] the weight of row lane/4 + 8i duplicated into both halves.  On exit
// x[2j + h] = sum over this thread's four rows of f_r e[r][8j + 2(lane%4) + h].
__device__ __forceinline__ void pass2_rows(const uint32_t (&a)[16], const uint32_t (&b)[16], const float2 (&fr2)[4], float (&x)[8])
{
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        float2 s = __ffma2_rn(fr2[0], make_float2(__uint_as_float(a[4 * j]), __uint_as_float(a[4 * j + 1])), make_float2(0.f, 0.f));
        s = __ffma2_rn(fr2[1], make_float2(__uint_as_float(a[4 * j + 2]), __uint_as_float(a[4 * j + 3])), s);
        s = __ffma2_rn(fr2[2], make_float2(__uint_as_float(b[4 * j]), __uint_as_float(b[4 * j + 1])), s);
        s = __ffma2_rn(fr2[3], make_float2(__uint_as_float(b[4 * j + 2]), __uint_as_float(b[4 * j + 3])), s);
        x[2 * j] = s.x;
        x[2 * j + 1] = s.y;
    }
}

// Adds the partial sums of the eight lanes that share lane % 4: on entry lane (g, p) = (lane / 4, lane % 4) holds
// x[2c + h] = its partial of column 8c + 2p + h (c < 4, h < 2); on exit it holds the complete sum of column
// 8 (g / 2) + 2p + (g % 2).  Three exchange steps, each halving the values a lane carries.
__device__ __forceinline__ float pass2_reduce(float (&x)[8], int lane)
{
    const bool up4 = lane & 16, up2 = lane & 8, up1 = lane & 4;
#pragma unroll
    for (int i = 0; i < 4; ++i) {  // g bit 2 picks x[4..7] or x[0..3]
        const float keep = up4 ? x[i + 4] : x[i], give = up4 ? x[i] : x[i + 4];
        x[i] = keep + __shfl_xor_sync(0xffffffffu, give, 16);
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {  // g bit 1 picks x[2..3] or x[0..1]
        const float keep = up2 ? x[i + 2] : x[i], give = up2 ? x[i] : x[i + 2];
        x[i] = keep + __shfl_xor_sync(0xffffffffu, give, 8);
    }
    const float keep = up1 ? x[1] : x[0], give = up1 ? x[0] : x[1];
    return keep + __shfl_xor_sync(0xffffffffu, give, 4);
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128
// bytes, 8-row groups 1024 bytes apart (the layout TMA writes with SWIZZLE_128B).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Instruction descriptor: D = fp32, A = B = bf16, both K-major, M = 128, N = 128 (one column half).
constexpr uint32_t kTcIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

// ------------------------------------------------------------------ the kernel
__global__ void __launch_bounds__(kTcThreads, 1)
cap_score_tc_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                    const __grid_constant__ CUtensorMap mapKnew, TcParams prm)
{
    extern __shared__ __align__(1024) uint8_t tc_smem_raw[];
    const uint32_t base = smem_u32(tc_smem_raw);
    if (base & 1023u) {  // the swizzled tiles need this alignment; nothing has been started yet
        if (threadIdx.x == 0) set_status(prm.status, kStatusBounds);
        return;
    }
    uint8_t *gbase = tc_smem_raw;
    uint32_t &tmem_base_slot = *reinterpret_cast<uint32_t *>(gbase + kTcOffTmemSlot);
    int &abort_flag = *reinterpret_cast<int *>(gbase + kTcOffAbort);
    const uint32_t bar0 = base + kTcOffBar;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        *reinterpret_cast<unsigned long long *>(gbase + kTcOffAbort + 4) = global_ns() + prm.wait_ns;
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar(kBarFull + b), 1);
            mbar_init(bar(kBarEmpty + b), 1);
            mbar_init(bar(kBarEReady + b), 512);
            mbar_init(bar(kBarFReady + b), 128);
            for (int h = 0; h < 2; ++h) {
                mbar_init(bar(kBarSFull + 2 * b + h), 1);
                mbar_init(bar(kBarTEmpty + 2 * b + h), 512);
            }
        }
        mbar_init(bar(kBarDrain), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {  // tensor memory: two buffers of 256 columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;
    volatile int *ab = &abort_flag;
    const int tasks_per_item = prm.slabs;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            uint32_t k = 0;
            for (int task = blockIdx.x; task < prm.tasks; task += gridDim.x, ++k) {
                const int item = task / tasks_per_item, slab = task - item * tasks_per_item;
                const int unit = item / prm.mtiles, mt = item - unit * prm.mtiles;
                const uint32_t b = k & 1, ph = (k >> 1) & 1;
                if (!mbar_wait(bar(kBarEmpty + b), ph ^ 1, ab, prm.status)) break;   // nothing more is put in flight
                mbar_expect_tx(bar(kBarFull + b), (uint32_t)prm.dhalves * (kTcStageBytes / 2));
                const uint32_t q = base + kTcOffStage + b * kTcStageBytes, kk = q + kTcQBytes;
                const bool fresh_rows = slab >= prm.new_slab0;
                const CUtensorMap *mk = fresh_rows ? &mapKnew : &mapK;
                const int krow = (fresh_rows ? slab - prm.new_slab0 : slab) * kTcSlab;
                tma_load_3d(q, &mapQ, 0, mt * kTcRows, unit, bar(kBarFull + b));
                tma_load_3d(kk, mk, 0, krow, unit, bar(kBarFull + b));
                if (prm.dhalves == 2) {
                    tma_load_3d(q + kTcQBytes / 2, &mapQ, 64, mt * kTcRows, unit, bar(kBarFull + b));
                    tma_load_3d(kk + kTcKBytes / 2, mk, 64, krow, unit, bar(kBarFull + b));
                }
            }
            // loads that were issued land in this CTA's shared memory: see the last one of either stage complete before
            // the CTA may end (k loads were issued; load j went to stage j & 1 as its (j >> 1)-th fill)
            for (uint32_t j = (k > 2 ? k - 2 : 0); j < k; ++j)
                mbar_wait(bar(kBarFull + (j & 1)), (j >> 1) & 1, ab, prm.status, false);
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            uint32_t k = 0;
            for (int task = blockIdx.x; task < prm.tasks; task += gridDim.x, ++k) {
                const uint32_t b = k & 1, ph = (k >> 1) & 1;
                if (!mbar_wait(bar(kBarFull + b), ph, ab, prm.status)) break;
                const uint32_t qa = base + kTcOffStage + b * kTcStageBytes, kb = qa + kTcQBytes;
                for (uint32_t h = 0; h < 2; ++h) {
                    if (!mbar_wait(bar(kBarTEmpty + 2 * b + h), ph ^ 1, ab, prm.status)) break;
                    tc_fence_after();
                    for (uint32_t blk = 0; blk < (uint32_t)prm.dhalves; ++blk) {
#pragma unroll
                        for (uint32_t k4 = 0; k4 < 4; ++k4) {
                            const uint32_t off = k4 * 32;
                            tc_mma_bf16(tmem + b * kTcSlab + h * 128, smem_desc_sw128(qa + blk * (kTcQBytes / 2) + off),
                                        smem_desc_sw128(kb + blk * (kTcKBytes / 2) + h * (128 * 128) + off), kTcIdesc,
                                        (blk | k4) ? 1u : 0u);
                        }
                    }
                    tc_commit(bar(kBarSFull + 2 * b + h));   // this half's logits are complete
                }
                if (*ab) break;
                tc_commit(bar(kBarEmpty + b));               // the stage may be refilled once the MMAs have read it
            }
            if (k) {  // every MMA has finished (and read its operands) before tensor memory is released
                tc_commit(bar(kBarDrain));
                mbar_wait(bar(kBarDrain), 0, ab, prm.status, false);
            }
        }
        __syncwarp();
    } else if (warp < 18) {
        // ---------------------------------------------------------------- pass 1 / pass 2 (512 threads)
        const int q = warp & 3;                 // TMEM lane quarter this warp may touch
        const int w = warp - 2;                 // 0..15
        const int cq = w >> 2;                  // this warp's columns: [32 cq, 32 cq + 32) of each buffer half
        const int row = q * 32 + lane;
        float2 *tstat = reinterpret_cast<float2 *>(gbase + kTcOffTstat);
        const float *fbuf = reinterpret_cast<const float *>(gbase + kTcOffFbuf);
        float *colpart = reinterpret_cast<float *>(gbase + kTcOffColpart);
        const float c = prm.scale_log2e;
        const int n_local = (prm.tasks - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
        for (int k = 0; k <= n_local; ++k) {
            if (k < n_local) {
                // ---- pass 1 of local task k
                const int task = blockIdx.x + k * gridDim.x;
                const int slab = task % tasks_per_item;
                const int nvalid = min(kTcSlab, prm.N - slab * kTcSlab);
                const uint32_t b = k & 1, ph = (k >> 1) & 1;
                const uint32_t t0 = tmem + ((uint32_t)(q * 32) << 16) + b * kTcSlab + cq * 32;
                if (nvalid == kTcSlab) {
                    // two chunks of 32 columns (one per buffer half) in four pieces of 16 through two register sets:
                    // the second half's first piece is fetched while the first half's second piece is still being
                    // exponentiated, so that its tensor-memory latency is not waited for
                    uint32_t X[16], Y[16];
                    mbar_wait(bar(kBarSFull + 2 * b), ph, ab, prm.status);
                    tc_fence_after();
                    tmem_ld16(t0, X);
                    tmem_ld16(t0 + 16, Y);
                    tmem_wait_ld16(X);
                    tmem_wait_ld16(Y);
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                        piece_max(X, mx);
                        piece_max(Y, mx);
                        const float mxc = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * c;
                        float2 sum[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                        piece_exp<0>(X, c, mxc, sum);
                        tmem_st16(t0 + h * 128, X);
                        // the second half's logits: fetched behind the next piece's exponentials if the tensor core has
                        // delivered them by now (lane 0's answer for the whole warp: a phase that is complete stays complete)
                        const bool early = h == 0 && __shfl_sync(0xffffffffu, mbar_test_wait(bar(kBarSFull + 2 * b + 1), ph) ? 1 : 0, 0);
                        if (early) {
                            tc_fence_after();
                            tmem_ld16(t0 + 128, X);
                        }
                        piece_exp<8>(Y, c, mxc, sum);
                        tmem_st16(t0 + h * 128 + 16, Y);
                        if (h == 0) {
                            if (!early) {
                                mbar_wait(bar(kBarSFull + 2 * b + 1), ph, ab, prm.status);
                                tc_fence_after();
                                tmem_ld16(t0 + 128, X);
                            }
                            tmem_ld16(t0 + 128 + 16, Y);
                        }
                        const float2 s01 = __fadd2_rn(sum[0], sum[1]), s23 = __fadd2_rn(sum[2], sum[3]);
                        tstat[(b * 8 + h * 4 + cq) * kTcRows + row] = make_float2(mxc, (s01.x + s01.y) + (s23.x + s23.y));
                        if (h == 0) {
                            tmem_wait_ld16(X);
                            tmem_wait_ld16(Y);
                        }
                    }
                } else {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        mbar_wait(bar(kBarSFull + 2 * b + h), ph, ab, prm.status);
                        tc_fence_after();
                        tstat[(b * 8 + h * 4 + cq) * kTcRows + row] = pass1_chunk<false>(t0 + h * 128, h * 128 + cq * 32, nvalid, c);
                    }
                }
                tmem_wait_st();
                tc_fence_before();  // pass 2 reads these TMEM words from other lanes of the warp
                mbar_arrive(bar(kBarEReady + b));
            }
            if (k >= 1) {
                // ---- pass 2 of local task k - 1
                const int kk = k - 1;
                const int task = blockIdx.x + kk * gridDim.x;
                const int item = task / tasks_per_item, slab = task - item * tasks_per_item;
                const int unit = item / prm.mtiles, mt = item - unit * prm.mtiles;
                const int nvalid = min(kTcSlab, prm.N - slab * kTcSlab);
                const uint32_t b = kk & 1, ph = (kk >> 1) & 1;
                const uint32_t trow = tmem + ((uint32_t)(q * 32) << 16) + b * kTcSlab + cq * 32;
                mbar_wait(bar(kBarFReady + b), ph, ab, prm.status);
                tc_fence_after();
                float *cpart = colpart + (kk & 1) * (4 * kTcSlab);
#pragma unroll
                for (int h = 0; h < 2; ++h) {  // this warp's 32 columns of buffer half h
                    float2 fr2[4];  // the weights of rows lane/4 + 8i for this chunk, duplicated for the packed FMAs
                    {
                        const float *f = fbuf + (b * 8 + h * 4 + cq) * kTcRows + q * 32 + (lane >> 2);
#pragma unroll
                        for (int i = 0; i < 4; ++i) fr2[i] = make_float2(f[8 * i], f[8 * i]);
                    }
                    float x[8];
                    uint32_t va[16], vb[16];
                    tmem_ld_16x256b_x4(trow + h * 128, va);
                    tmem_ld_16x256b_x4(trow + h * 128 + (16u << 16), vb);
                    tmem_wait_ld16(va);
                    tmem_wait_ld16(vb);
                    tc_fence_before();
                    mbar_arrive(bar(kBarTEmpty + 2 * b + h));   // this half may be overwritten by the task after next
                    pass2_rows(va, vb, fr2, x);
                    const float u = pass2_reduce(x, lane);
                    const int g = lane >> 2, pp = lane & 3;
                    cpart[q * kTcSlab + h * 128 + cq * 32 + 8 * (g >> 1) + 2 * pp + (g & 1)] = u;
                }
                // ---- add the four row quarters of this column group, store its 64 scores
                column_group_sync(cq);
                if (q < 2) {  // warp q = 0 stores the group's columns of half 0, warp q = 1 those of half 1
                    const int col = q * 128 + cq * 32 + lane;
                    if (col < nvalid) {
                        float *out = prm.scores + (size_t)mt * prm.part_stride + (size_t)unit * prm.N + slab * kTcSlab;
                        out[col] = (cpart[col] + cpart[kTcSlab + col]) + (cpart[2 * kTcSlab + col] + cpart[3 * kTcSlab + col]);
                    }
                }
                // no second barrier: the next task writes the other parity of colpart, and the one after
                // that is separated from these reads by the next task's barrier
            }
        }
    } else {
        // ---------------------------------------------------------------- combine (128 threads, one per query row)
        const int row = threadIdx.x - 576;
        const float2 *tstat = reinterpret_cast<const float2 *>(gbase + kTcOffTstat);
        float *fbuf = reinterpret_cast<float *>(gbase + kTcOffFbuf);
        const float sgn = prm.sign;
        uint32_t k = 0;
        for (int task = blockIdx.x; task < prm.tasks; task += gridDim.x, ++k) {
            const int item = task / tasks_per_item, slab = task - item * tasks_per_item;
            const int mt = item % prm.mtiles;
            const uint32_t b = k & 1, ph = (k >> 1) & 1;
            const bool row_valid = mt * kTcRows + row < prm.M;
            float2 own = make_float2(-INFINITY, 0.f);  // the CaP keys' share of this row's denominator (Appendix B listing)
            if (prm.cap_stats && row_valid) own = __ldg(&prm.cap_stats[(size_t)(item / prm.mtiles) * prm.M + mt * kTcRows + row]);
            mbar_wait(bar(kBarEReady + b), ph, ab, prm.status);
            // ---- merge the eight chunks of the row, publish the slab's statistics
            // (this warp shares its scheduler with four busy epilogue warps and every task waits for this code: the
            // loads are issued together and maxima and sums are folded as trees, not as chains)
            float cm[8], ce[8];
            {
                float2 t[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) t[i] = tstat[(b * 8 + i) * kTcRows + row];
#pragma unroll
                for (int i = 0; i < 8; ++i) cm[i] = t[i].x;
                const float ms0 = max3(max3(cm[0], cm[1], cm[2]), max3(cm[3], cm[4], cm[5]), fmaxf(cm[6], cm[7]));  // chunk 0 always holds a valid key
#pragma unroll
                for (int i = 0; i < 8; ++i) ce[i] = (cm[i] == -INFINITY) ? 0.f : t[i].y * ex2(cm[i] - ms0);
            }
            const float ms = max3(max3(cm[0], cm[1], cm[2]), max3(cm[3], cm[4], cm[5]), fmaxf(cm[6], cm[7]));
            const float ls = ((ce[0] + ce[1]) + (ce[2] + ce[3])) + ((ce[4] + ce[5]) + (ce[6] + ce[7]));
            if (tasks_per_item > 1 && (int)blockIdx.x != prm.withhold_cta) st_gpu_f32x2(&prm.stats[((size_t)item * tasks_per_item + slab) * kTcRows + row], ms, ls * sgn);

            // ---- this row's statistics of every slab of the item; re-read until all carry this launch's mark
            const float2 *st = prm.stats + (size_t)item * tasks_per_item * kTcRows + row;
            float m = -INFINITY, l = 0.f;
            if (tasks_per_item == 1) {  // the item is this slab: nothing to exchange
                m = ms;
                l = ls;
            }
            for (int s0 = 0; s0 < (tasks_per_item > 1 ? tasks_per_item : 0); s0 += 16) {
                float2 sv[16];
                uint32_t tries = 0;
                bool fresh;
#pragma unroll
                for (int s = 0; s < 16; ++s)  // beyond the item: neutral and fresh; this CTA's own slab: known; others: stale
                    sv[s] = (s0 + s >= tasks_per_item) ? make_float2(-INFINITY, sgn) : (s0 + s == slab) ? make_float2(ms, ls * sgn) : make_float2(0.f, 0.f);
                do {  // only the entries that are still stale are read again
                    fresh = true;
#pragma unroll
                    for (int s = 0; s < 16; ++s) {
                        if (!(sv[s].y * sgn > 0.f)) sv[s] = ld_gpu_f32x2(&st[(size_t)(s0 + s) * kTcRows]);
                        fresh = fresh && (sv[s].y * sgn > 0.f);
                    }
                    if (!fresh && (*ab || ((++tries & 1023u) == 0 && global_ns() > *reinterpret_cast<volatile unsigned long long *>(ab + 1)))) {
                        if (!*ab) {
                            *ab = 1;
                            set_status(prm.status, kStatusTimeout);
                        }
                        break;
                    }
                } while (!fresh);
                const float mb = max3(max3(max3(sv[0].x, sv[1].x, sv[2].x), max3(sv[3].x, sv[4].x, sv[5].x), max3(sv[6].x, sv[7].x, sv[8].x)),
                                      max3(max3(sv[9].x, sv[10].x, sv[11].x), max3(sv[12].x, sv[13].x, sv[14].x), fmaxf(sv[15].x, m)), -INFINITY);
                float w[16];
#pragma unroll
                for (int s = 0; s < 16; ++s) w[s] = fabsf(sv[s].y) * ex2(sv[s].x - mb);
#pragma unroll
                for (int step = 1; step < 16; step <<= 1) {
#pragma unroll
                    for (int s = 0; s < 16; s += 2 * step) w[s] += w[s + step];
                }
                l = ((m == -INFINITY) ? 0.f : l * ex2(m - mb)) + w[0];
                m = mb;
            }
            if (own.x > -INFINITY) {
                const float mb = fmaxf(m, own.x);
                l = fmaf(own.y, ex2(own.x - mb), l * ex2(m - mb));
                m = mb;
            }
            float inv_l;
            asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv_l) : "f"(l));
            if (!row_valid) inv_l = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i)
                fbuf[(b * 8 + i) * kTcRows + row] = (cm[i] == -INFINITY) ? 0.f : ex2(cm[i] - m) * inv_l;
            mbar_arrive(bar(kBarFReady + b));
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*TcEncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                               const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TcPlan {
    bool usable = false;
    TcEncodeFn encode = nullptr;
    int sm_count = 0;
    int max_items = 0, max_slabs = 0;
    float2 *stats = nullptr;          // [max_items][max_slabs][128]
    // "fresh" marking of the statistics: every launch writes all entries of its (items x slabs) layout
    // with the sign opposite to the previous launch's; a layout change clears the array first
    float sign = 1.f;
    int last_items = 0, last_slabs = 0;
};

inline void tc_plan_destroy(TcPlan &plan)
{
    cudaFree(plan.stats);
    plan.stats = nullptr;
    plan.usable = false;
}

inline void tc_plan_init(TcPlan &plan, const ipot_config_t &cfg, const void *, int sm_count)
{
    plan.usable = false;
    plan.sm_count = sm_count;
    if (cfg.dtype != IPOT_BF16 || (cfg.d != 128 && cfg.d != 64)) return;
    int coop = 0, dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) {
        cudaGetLastError();
        return;
    }
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn) {
        cudaGetLastError();
        return;
    }
    plan.encode = reinterpret_cast<TcEncodeFn>(fn);
    if (cudaFuncSetAttribute(cap_score_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcSmemBytes) != cudaSuccess) {
        cudaGetLastError();
        return;
    }
    const int G = cfg.Hq / cfg.Hkv;
    const int units = cfg.layers * cfg.batch * cfg.Hkv;
    plan.max_items = units * ((G * cfg.max_cap_rows + kTcRows - 1) / kTcRows);
    plan.max_slabs = (cfg.pot_size + kTcSlab - 1) / kTcSlab;
    if (cudaMalloc(&plan.stats, (size_t)plan.max_items * plan.max_slabs * kTcRows * sizeof(float2)) != cudaSuccess) {
        cudaGetLastError();
        tc_plan_destroy(plan);
        return;
    }
    plan.usable = true;
}

inline bool tc_applicable(TcPlan &plan, const ipot_config_t &cfg, int N, int M)
{
    if (!plan.usable || cfg.dtype != IPOT_BF16 || (cfg.d != 128 && cfg.d != 64) || N < 1 || M < 1) return false;
    const int units = cfg.layers * cfg.batch * cfg.Hkv;
    return units * ((M + kTcRows - 1) / kTcRows) <= plan.max_items && (N + kTcSlab - 1) / kTcSlab <= plan.max_slabs;
}

// [units][unit_rows][d] bf16, of which `rows` per unit are addressable; box = 64 x box_rows x 1, 128-byte swizzle.
inline int tc_encode_rows(TcPlan &plan, CUtensorMap *map, const void *ptr, int d, int rows, int units, size_t unit_rows, int box_rows)
{
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)rows, (cuuint64_t)units};
    cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)unit_rows * d * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = plan.encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? IPOT_OK : IPOT_E_CUDA;
}

// scores: partial array p (query rows 128 p ...) is written at scores + p * part_stride, unit stride N.
// Knew (may be NULL): the keys from slot new_first on are not in the pot yet but in this [units][N - new_first][d]
// array (the chunk of a deferred append); new_first must be a multiple of the slab size.
inline int tc_launch(TcPlan &plan, const ipot_config_t &cfg, const void *Q, const void *K, const float2 *cap_stats, float *scores,
                     size_t part_stride, int N, int M, int units, int *status, cudaStream_t stream, int *parts, int *n_launch,
                     const void *Knew = nullptr, int new_first = 0, unsigned long long wait_ns = 200ull * 1000 * 1000,
                     int withhold_cta = -1, int spare_sms = 0)
{
    if (!tc_applicable(plan, cfg, N, M)) return IPOT_E_INVALID;
    if (Knew && (new_first % kTcSlab != 0 || new_first >= N)) return IPOT_E_INVALID;
    const int mtiles = (M + kTcRows - 1) / kTcRows;
    CUtensorMap mapQ, mapK, mapKnew;
    if (tc_encode_rows(plan, &mapQ, Q, cfg.d, M, units, (size_t)M, kTcRows) != IPOT_OK) return IPOT_E_CUDA;
    if (Knew && new_first == 0) {  // every key is in the chunk
        if (tc_encode_rows(plan, &mapK, Knew, cfg.d, N, units, (size_t)N, kTcSlab) != IPOT_OK) return IPOT_E_CUDA;
        Knew = nullptr;
    } else if (tc_encode_rows(plan, &mapK, K, cfg.d, Knew ? new_first : N, units, (size_t)cfg.pot_size, kTcSlab) != IPOT_OK) {
        return IPOT_E_CUDA;
    }
    if (!Knew) mapKnew = mapK;
    else if (tc_encode_rows(plan, &mapKnew, Knew, cfg.d, N - new_first, units, (size_t)(N - new_first), kTcSlab) != IPOT_OK) return IPOT_E_CUDA;
    TcParams prm;
    prm.scores = scores; prm.part_stride = part_stride; prm.stats = plan.stats; prm.cap_stats = cap_stats; prm.status = status;
    prm.N = N; prm.M = M; prm.mtiles = mtiles; prm.slabs = (N + kTcSlab - 1) / kTcSlab;
    const int items = units * mtiles;
    prm.tasks = items * prm.slabs;
    prm.dhalves = cfg.d / 64;
    prm.new_slab0 = Knew ? new_first / kTcSlab : 0x7fffffff;
    prm.scale_log2e = (float)(1.4426950408889634 / sqrt((double)cfg.d));
    prm.wait_ns = wait_ns;
    prm.withhold_cta = withhold_cta;
    if (items != plan.last_items || prm.slabs != plan.last_slabs) {
        if (cudaMemsetAsync(plan.stats, 0, (size_t)items * prm.slabs * kTcRows * sizeof(float2), stream) != cudaSuccess) {
            cudaGetLastError();
            return IPOT_E_CUDA;
        }
        plan.last_items = items;
        plan.last_slabs = prm.slabs;
    }
    plan.sign = -plan.sign;
    prm.sign = plan.sign;
    cudaLaunchConfig_t lc = {};
    // spare_sms: SMs left to a small kernel of the same cycle that runs beside this one on another stream
    const int ctas = plan.sm_count - spare_sms > 0 ? plan.sm_count - spare_sms : 1;
    lc.gridDim = dim3(prm.tasks < ctas ? prm.tasks : ctas, 1, 1);
    lc.blockDim = dim3(kTcThreads, 1, 1);
    lc.dynamicSmemBytes = kTcSmemBytes;
    lc.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeCooperative;  // all CTAs resident: they wait on each other's statistics
    at[0].val.cooperative = 1;
    lc.attrs = at; lc.numAttrs = 1;
    if (cudaLaunchKernelEx(&lc, cap_score_tc_kernel, mapQ, mapK, mapKnew, prm) != cudaSuccess) {
        cudaGetLastError();
        return IPOT_E_CUDA;
    }
    *parts = mtiles;
    *n_launch = 1;
    return IPOT_OK;
}

}  // namespace ipotk
