// Host side of the memory-pot library: pot state, argument checks, launches.
// The C ABI is declared and documented in include/ipot.h.
#include "../../include/ipot.h"

#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>

#include "common.cuh"
#include "k_cap_self.cuh"
#include "k_decode.cuh"
#include "k_move.cuh"
#include "k_novelty.cuh"
#include "k_rope.cuh"
#include "k_score_mma.cuh"
#include "k_score_simt.cuh"
#include "k_score_tc.cuh"
#include "k_score_ts.cuh"
#include "k_select.cuh"

using namespace ipotk;

struct ipot {
    ipot_config_t cfg;
    int len;
    int device;
    int sm_count;
    int scorer;
    int G, units, elem_bytes, row_bytes;
    int compact_slices, rope_slices;
    cudaStream_t stream;
    // Deferred append (ipot_set_deferred_append): the newest chunk's rows (slots pend_first .. len - 1) still lie in
    // the caller's buffers; the tensor-core scorer reads its keys there and the compaction fetches the survivors
    // from there, so rows that the cycle drops are never copied.  NULL = those rows are in the pot.
    int deferred;
    const void *pend_K, *pend_V;
    int pend_n, pend_first;
    // device memory (library-owned)
    void *K, *V;
    // CR-RoPE (ipot_enable_rope): K then holds the keys without rotary embedding, Krot the copy rotated at the slot
    // numbers, which is what the scorers read; the tables are the caller's
    void *Krot;
    const void *rope_cos, *rope_sin;
    int rope;            // 0 off, IPOT_ROPE_HALF, IPOT_ROPE_INTERLEAVED
    float *scores;       // [max_parts][units * pot_size]; array q holds [units][N] partial scores of the
                         // q-th block of 128 query rows (the SIMT scorer writes array 0 only)
    float *summed;       // [units][N]: sum of the partial arrays when there are several
    int max_parts;
    float2 *row_stats;   // [units][max M]
    float2 *mma_part;    // [kMmaSplits][units][max M]: partial row statistics of the warp-level tensor-core scorer
    float2 *cap_stats;   // [units][max M]: (max, sum) over the CaP's own keys, CaP-inclusive scoring only
    uint8_t *nuc_mask;   // [batch][pot_size]
    int32_t *idx;        // [units][keep]
    int *status;         // sticky device status word
    void *stage_q;       // device staging for the *_host calls
    void *stage_kc;
    float *dec_partial;  // [units][dec_splits][G][d + 2]: ipot_decode_attention's split results
    int *dec_counters;   // [units], zero between calls
    int dec_splits;
    char *nov_scratch;   // scratch of ipot_nuc_scores, grown on demand: 65536 row counters (always zero between
                         // calls), then [tokens][segments] float2
    size_t nov_capacity;  // float2 entries behind the counters
    float *stage_aux;
    // results of the last cycle
    int last_len_before;
    const float *last_scores;
    int last_scorer;
    // timing
    int profiling;
    cudaEvent_t (*ev)[5];  // kProfSlots event quintuples, one per recorded cycle
    int ev_used;
    long long launches;
    TcPlan tc;           // tensor-core scorer state
    TsTuning ts;         // launch parameters of the two-sweep tensor-core scorer
    TsOccupancy ts_occ;
    // the novelty ranking does not depend on the scores: it runs beside the scorer on a stream of its own
    cudaStream_t side;
    cudaEvent_t ev_fork, ev_join;
};

namespace {

constexpr int kProfSlots = 2048;
constexpr int kMmaSplits = 8;
constexpr size_t kNovCounterBytes = (size_t)(kNovMaxRows + 1) * sizeof(int);

#define IPOT_CUDA(call)                                                             \
    do {                                                                            \
        cudaError_t e_ = (call);                                                    \
        if (e_ != cudaSuccess) {                                                    \
            if (getenv("IPOT_DEBUG"))                                               \
                fprintf(stderr, "ipot: %s -> %s\n", #call, cudaGetErrorString(e_)); \
            return IPOT_E_CUDA;                                                     \
        }                                                                           \
    } while (0)

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// the keys the CaP queries attend to
const void *score_keys(const ipot *p) { return p->rope ? p->Krot : p->K; }

int check_config(const ipot_config_t &c)
{
    if (c.pot_size <= 0 || c.pot_size > 32768) return IPOT_E_INVALID;
    if (c.keep <= 0 || c.keep >= c.pot_size) return IPOT_E_INVALID;
    if (c.layers <= 0 || c.batch <= 0 || c.Hq <= 0 || c.Hkv <= 0 || c.Hq % c.Hkv) return IPOT_E_INVALID;
    if (c.d < 32 || c.d > 256 || c.d % 8) return IPOT_E_INVALID;
    if (c.dtype != IPOT_BF16 && c.dtype != IPOT_F32) return IPOT_E_INVALID;
    if (c.nuc_slots < -1 || c.nuc_slots > c.keep) return IPOT_E_INVALID;
    if (c.max_cap_rows <= 0 || c.max_cap_rows > 4096) return IPOT_E_INVALID;
    return IPOT_OK;
}

void free_all(ipot *p)
{
    tc_plan_destroy(p->tc);
    cudaFree(p->K); cudaFree(p->V); cudaFree(p->Krot); cudaFree(p->scores); cudaFree(p->summed);
    cudaFree(p->row_stats); cudaFree(p->mma_part); cudaFree(p->cap_stats); cudaFree(p->nuc_mask); cudaFree(p->idx); cudaFree(p->status);
    cudaFree(p->stage_q); cudaFree(p->stage_kc); cudaFree(p->stage_aux); cudaFree(p->nov_scratch); cudaFree(p->dec_partial); cudaFree(p->dec_counters);
    if (p->ev_fork) cudaEventDestroy(p->ev_fork);
    if (p->ev_join) cudaEventDestroy(p->ev_join);
    if (p->side) cudaStreamDestroy(p->side);
    if (p->ev) {
        for (int i = 0; i < kProfSlots; ++i)
            for (auto &e : p->ev[i]) if (e) cudaEventDestroy(e);
        delete[] p->ev;
    }
}

// Copies the rows of a deferred append that are still in the caller's buffers into the pot (keys, values or both).
int materialise(ipot *p, bool keys, bool values)
{
    const void *k = keys ? p->pend_K : nullptr, *v = values ? p->pend_V : nullptr;
    if (!k && !v) return IPOT_OK;
    const size_t row_vecs = p->row_bytes / 16, n_vecs = (size_t)p->pend_n * row_vecs;
    int pieces = (int)((n_vecs + (size_t)kMoveThreads * kMoveVecs - 1) / ((size_t)kMoveThreads * kMoveVecs));
    if (pieces < 1) pieces = 1;
    dim3 grid(pieces, p->units, (k && v) ? 2 : 1);
    if (k && v)
        append_kernel<<<grid, kMoveThreads, 0, p->stream>>>((const uint4 *)k, (const uint4 *)v, (uint4 *)p->K, (uint4 *)p->V, n_vecs,
                                                           (size_t)p->cfg.pot_size * row_vecs, (size_t)p->pend_first * row_vecs);
    else
        append_kernel<<<grid, kMoveThreads, 0, p->stream>>>((const uint4 *)(k ? k : v), nullptr, (uint4 *)(k ? p->K : p->V), nullptr, n_vecs,
                                                           (size_t)p->cfg.pot_size * row_vecs, (size_t)p->pend_first * row_vecs);
    p->launches += 1;
    IPOT_CUDA(cudaGetLastError());
    if (k) p->pend_K = nullptr;
    if (v) p->pend_V = nullptr;
    return IPOT_OK;
}

PendingRows pending_rows(const ipot *p)
{
    PendingRows r;
    r.K = (const uint4 *)p->pend_K;
    r.V = (const uint4 *)p->pend_V;
    r.unit_vecs = (size_t)p->pend_n * (p->row_bytes / 16);
    r.first = p->pend_first;
    return r;
}

// Row statistics over the CaP's own keys (causal): what Appendix B's listing adds to every row's denominator.
int launch_cap_self(ipot *p, const void *Q, const void *Kc, int M, int P)
{
    const int d = p->cfg.d;
    const float scale_log2e = (float)(1.4426950408889634 / std::sqrt((double)d));
    if (p->cfg.dtype == IPOT_BF16 && d % 16 == 0) {
        dim3 g((M + kSelfRows - 1) / kSelfRows, p->units);
        cap_self_stats_bf16<<<g, kSelfWarps * 32, self_smem_bytes(d), p->stream>>>((const __nv_bfloat16 *)Q, (const __nv_bfloat16 *)Kc, p->cap_stats,
                                                                 M, P, d, scale_log2e);
    } else {
        dim3 g((M + kSimtRows - 1) / kSimtRows, p->units);
        if (p->cfg.dtype == IPOT_F32)
            cap_row_stats<float><<<g, kSimtThreads, simt_smem_bytes(d), p->stream>>>(
                (const float *)Q, (const float *)Kc, p->cap_stats, M, P, d, (size_t)P * d, scale_log2e, nullptr, P, 0);
        else
            cap_row_stats<__nv_bfloat16><<<g, kSimtThreads, simt_smem_bytes(d), p->stream>>>(
                (const __nv_bfloat16 *)Q, (const __nv_bfloat16 *)Kc, p->cap_stats, M, P, d, (size_t)P * d, scale_log2e, nullptr, P, 0);
    }
    p->launches += 1;
    IPOT_CUDA(cudaGetLastError());
    return IPOT_OK;
}

template <typename T>
int launch_simt(ipot *p, const void *Q, const float2 *cap_stats, int M, int N)
{
    const int d = p->cfg.d;
    const size_t smem = simt_smem_bytes(d);
    const float scale_log2e = (float)(1.4426950408889634 / std::sqrt((double)d));
    const size_t kstride = (size_t)p->cfg.pot_size * d;
    dim3 g1((M + kSimtRows - 1) / kSimtRows, p->units), g2((N + kSimtKeys - 1) / kSimtKeys, p->units);
    cap_row_stats<T><<<g1, kSimtThreads, smem, p->stream>>>((const T *)Q, (const T *)score_keys(p), p->row_stats, M, N, d, kstride, scale_log2e,
                                                            cap_stats, 0, 1);
    cap_column_sums<T><<<g2, kSimtThreads, smem, p->stream>>>((const T *)Q, (const T *)score_keys(p), p->row_stats, p->scores, M, N, d, kstride, scale_log2e);
    p->launches += 2;
    IPOT_CUDA(cudaGetLastError());
    return IPOT_OK;
}

// bf16 pots with d a multiple of 16 that the tcgen05 kernel does not take: the same two launches on warp-level tensor cores
int launch_warp_mma(ipot *p, const void *Q, const float2 *cap_stats, int M, int N)
{
    const int d = p->cfg.d;
    const size_t smem = mma_scorer_smem_bytes(d);
    const float scale_log2e = (float)(1.4426950408889634 / std::sqrt((double)d));
    const size_t kstride = (size_t)p->cfg.pot_size * d;
    const int row_tiles = (M + kMsRows - 1) / kMsRows;
    // the row pass splits the keys so that it launches about four blocks per SM (at most kMmaSplits splits of whole tiles)
    int nsplit = (4 * p->sm_count + row_tiles * p->units - 1) / (row_tiles * p->units);
    const int key_tiles = (N + kMsKeys - 1) / kMsKeys;
    if (nsplit > kMmaSplits) nsplit = kMmaSplits;
    if (nsplit > key_tiles) nsplit = key_tiles;
    if (nsplit < 1) nsplit = 1;
    const int per = ((key_tiles + nsplit - 1) / nsplit) * kMsKeys;
    dim3 g1(row_tiles, p->units, nsplit), g2(key_tiles, p->units);
    const __nv_bfloat16 *Qb = (const __nv_bfloat16 *)Q, *Kb = (const __nv_bfloat16 *)score_keys(p);
    cap_row_stats_mma<<<g1, kMsWarps * 32, smem, p->stream>>>(Qb, Kb, p->mma_part, M, N, d, kstride, scale_log2e, per);
    cap_column_sums_mma<<<g2, kMsWarps * 32, smem, p->stream>>>(Qb, Kb, p->mma_part, cap_stats, nsplit, p->scores, M, N, d, kstride,
                                                               scale_log2e);
    p->launches += 2;
    IPOT_CUDA(cudaGetLastError());
    return IPOT_OK;
}

// The fastest scorer the shape allows.
int auto_scorer(const ipot *p, int N, int M, bool tc_ok, bool ts_ok, bool mma_ok)
{
    (void)p;
    (void)N;
    // measured on the three-to-four-row-block shapes (M = 384, 512): the two-sweep kernel holds every query tile of a
    // unit against a key slab that is fetched once per sweep and is 1.4 x faster there; up to two row blocks the
    // one-sweep kernel with its statistics exchange is as fast or faster
    if (ts_ok && (!tc_ok || M > 2 * kTcRows)) return IPOT_SCORER_TENSOR_SWEEPS;
    if (tc_ok) return IPOT_SCORER_TENSOR;
    return mma_ok ? IPOT_SCORER_WARP_MMA : IPOT_SCORER_SIMT;
}

// Steps 1-2 (and the timing events around them).  On success *parts tells how many
// partial score arrays the scorer wrote.
int run_scoring(ipot *p, const void *Q, const void *Kc, int cap_rows, const float *aux, int *parts)
{
    const int N = p->len, T = p->cfg.nuc_slots, M = p->G * cap_rows;
    int scorer = p->scorer;
    const bool tc_ok = tc_applicable(p->tc, p->cfg, N, M);
    const bool ts_ok = ts_applicable(p->tc, p->cfg, N, M);
    const bool mma_ok = p->cfg.dtype == IPOT_BF16 && p->cfg.d % 16 == 0;
    if (scorer == IPOT_SCORER_TENSOR && !tc_ok) return IPOT_E_INVALID;
    if (scorer == IPOT_SCORER_TENSOR_SWEEPS && !ts_ok) return IPOT_E_INVALID;
    if (scorer == IPOT_SCORER_WARP_MMA && !mma_ok) return IPOT_E_INVALID;
    if (scorer == IPOT_SCORER_AUTO) scorer = auto_scorer(p, N, M, tc_ok, ts_ok, mma_ok);
    // keys of a deferred append: the tensor-core scorers read whole slabs of them where they are, anything else
    // wants them in the pot
    const int slab_keys = scorer == IPOT_SCORER_TENSOR ? kTcSlab : scorer == IPOT_SCORER_TENSOR_SWEEPS ? kTsSlab : 0;
    const bool keys_in_chunk = p->pend_K && slab_keys && p->pend_first % slab_keys == 0;
    if (p->pend_K && !keys_in_chunk) {
        int mrc = materialise(p, true, false);
        if (mrc != IPOT_OK) return mrc;
    }

    cudaEvent_t *ev = (p->profiling && p->ev_used < kProfSlots) ? p->ev[p->ev_used] : nullptr;
    if (ev) IPOT_CUDA(cudaEventRecord(ev[0], p->stream));
    // Sec. 3.3.3: the T most novel slots per stream.  One block per stream and independent of the scores, so it is
    // queued on the side stream (after everything the caller has queued so far) and the tensor-core scorers leave
    // it one SM; the selection waits for both.  Other scorers fill the device in waves and need no such care.
    const bool side_nuc = T > 0 && aux && p->side && (scorer == IPOT_SCORER_TENSOR || scorer == IPOT_SCORER_TENSOR_SWEEPS);
    if (T > 0 && aux) {
        cudaStream_t ns = side_nuc ? p->side : p->stream;
        if (side_nuc) {
            IPOT_CUDA(cudaEventRecord(p->ev_fork, p->stream));
            IPOT_CUDA(cudaStreamWaitEvent(p->side, p->ev_fork, 0));
        }
        launch_nuc_mask(p->cfg.batch, ns, aux, p->nuc_mask, N, T);
        p->launches += 1;
        IPOT_CUDA(cudaGetLastError());
        if (side_nuc) IPOT_CUDA(cudaEventRecord(p->ev_join, p->side));
    }
    if (ev) IPOT_CUDA(cudaEventRecord(ev[1], p->stream));
    *parts = 1;
    int rc;
    if (Kc) {
        rc = launch_cap_self(p, Q, Kc, M, cap_rows);
        if (rc != IPOT_OK) return rc;
    }
    const float2 *cap_stats = Kc ? p->cap_stats : nullptr;
    if (scorer == IPOT_SCORER_TENSOR) {
        int n_launch = 0;
        rc = tc_launch(p->tc, p->cfg, Q, score_keys(p), cap_stats, p->scores, (size_t)p->units * p->cfg.pot_size, N, M, p->units, p->status,
                       p->stream, parts, &n_launch, keys_in_chunk ? p->pend_K : nullptr, keys_in_chunk ? p->pend_first : 0, p->ts.wait_ns,
                       p->ts.withhold_rank, side_nuc ? 1 : 0);
        p->launches += n_launch;
    } else if (scorer == IPOT_SCORER_TENSOR_SWEEPS) {
        rc = ts_launch(p->tc, p->ts_occ, p->ts, p->cfg, Q, score_keys(p), cap_stats, p->scores, N, M, p->units, p->status, p->stream,
                       keys_in_chunk ? p->pend_K : nullptr, keys_in_chunk ? p->pend_first : 0, side_nuc ? 1 : 0);
        p->launches += 1;
    } else if (scorer == IPOT_SCORER_WARP_MMA) {
        rc = launch_warp_mma(p, Q, cap_stats, M, N);
    } else {
        rc = p->cfg.dtype == IPOT_F32 ? launch_simt<float>(p, Q, cap_stats, M, N) : launch_simt<__nv_bfloat16>(p, Q, cap_stats, M, N);
    }
    if (ev && rc == IPOT_OK) IPOT_CUDA(cudaEventRecord(ev[2], p->stream));   // the scorer's end, before the join below
    if (side_nuc) IPOT_CUDA(cudaStreamWaitEvent(p->stream, p->ev_join, 0));   // (also when the scorer refused: nothing is left behind on the side stream)
    if (rc != IPOT_OK) return rc;
    p->last_scorer = scorer;
    p->last_len_before = N;
    p->last_scores = (*parts > 1) ? p->summed : p->scores;
    return IPOT_OK;
}

int check_cycle_args(ipot *p, const void *Q, int cap_rows, const float *aux, bool compress)
{
    if (!p || !Q) return IPOT_E_INVALID;
    if (cap_rows < 1 || cap_rows > p->cfg.max_cap_rows) return IPOT_E_INVALID;
    if (compress && p->cfg.nuc_slots > 0 && !aux) return IPOT_E_INVALID;
    if (compress ? (p->len <= p->cfg.keep) : (p->len < 1)) return IPOT_E_STATE;
    return IPOT_OK;
}

// One launch: z = 0 gathers the unrotated keys and writes the rotated copy, z = 1 gathers the values.
template <typename T>
void launch_compact_rope_t(ipot *p, int keep, int N, int row_vecs, size_t unit_vecs)
{
    const int ks = p->rope_slices, vs = p->compact_slices;
    dim3 grid(ks > vs ? ks : vs, p->units, 2);
    auto kern = p->rope == IPOT_ROPE_INTERLEAVED ? compact_rope_kernel<T, true> : compact_rope_kernel<T, false>;
    kern<<<grid, kMoveThreads, 0, p->stream>>>((uint4 *)p->K, (uint4 *)p->Krot, (const T *)p->rope_cos, (const T *)p->rope_sin, p->idx,
                                               keep, N, row_vecs, ks, row_vecs / 2 / ks, unit_vecs, p->status, (uint4 *)p->V, vs,
                                               row_vecs / vs, pending_rows(p));
}

void launch_compact_rope(ipot *p, int keep, int N, int row_vecs, size_t unit_vecs)
{
    if (p->cfg.dtype == IPOT_F32) launch_compact_rope_t<float>(p, keep, N, row_vecs, unit_vecs);
    else launch_compact_rope_t<__nv_bfloat16>(p, keep, N, row_vecs, unit_vecs);
}

// New key rows (src, unit stride src_unit_vecs) -> pot rows [len, len + n) unrotated and rotated; if srcV is not
// NULL the same launch copies the value rows ([units][n rows]) into the pot.
template <typename T>
void launch_append_rope_t(ipot *p, const void *src, size_t src_unit_vecs, const void *srcV, int n)
{
    const int row_vecs = p->row_bytes / 16;
    const size_t items = (size_t)n * (row_vecs / 2), unit_vecs = (size_t)p->cfg.pot_size * row_vecs;
    int pieces = (int)((items + (size_t)kMoveThreads * 4 - 1) / ((size_t)kMoveThreads * 4));
    if (pieces < 1) pieces = 1;
    dim3 grid(pieces, p->units, srcV ? 2 : 1);
    auto kern = p->rope == IPOT_ROPE_INTERLEAVED ? append_rope_kernel<T, true> : append_rope_kernel<T, false>;
    kern<<<grid, kMoveThreads, 0, p->stream>>>((const uint4 *)src, src_unit_vecs, (uint4 *)p->K, (uint4 *)p->Krot, (const T *)p->rope_cos,
                                               (const T *)p->rope_sin, n, row_vecs, unit_vecs, p->len, (const uint4 *)srcV, (uint4 *)p->V);
}

void launch_append_rope(ipot *p, const void *src, size_t src_unit_vecs, const void *srcV, int n)
{
    if (p->cfg.dtype == IPOT_F32) launch_append_rope_t<float>(p, src, src_unit_vecs, srcV, n);
    else launch_append_rope_t<__nv_bfloat16>(p, src, src_unit_vecs, srcV, n);
}

// Byte-column slices per row for the compaction grid: enough blocks to fill the device, slices of >= 64 bytes.
int compact_slices(const ipot *p)
{
    const int row_vecs = p->row_bytes / 16;
    int slices = 1;
    while (row_vecs % (slices * 2) == 0 && row_vecs / (slices * 2) >= 4 &&
           (long long)p->units * 2 * slices < 8LL * p->sm_count)
        slices *= 2;
    return slices;
}

// The same for the vector pairs (g, g + row_vecs / 2) of compact_rope_kernel: slices of >= 2 pairs.
int rope_slices(const ipot *p)
{
    const int half_vecs = p->row_bytes / 32;
    int slices = 1;
    while (half_vecs % (slices * 2) == 0 && half_vecs / (slices * 2) >= 2 &&
           (long long)p->units * slices < 8LL * p->sm_count)
        slices *= 2;
    return slices;
}

int run_cycle(ipot *p, const void *Q, const void *Kc, int cap_rows, const float *aux)
{
    const int N = p->len, keep = p->cfg.keep, T = p->cfg.nuc_slots;
    int parts = 1;
    cudaEvent_t *ev = (p->profiling && p->ev_used < kProfSlots) ? p->ev[p->ev_used] : nullptr;
    int rc = run_scoring(p, Q, Kc, cap_rows, aux, &parts);
    if (rc != IPOT_OK) return rc;
    const size_t part_stride = (size_t)p->units * p->cfg.pot_size;
    launch_select(p->units, p->stream, p->scores, parts, part_stride, T > 0 ? p->nuc_mask : nullptr, p->idx,
                  parts > 1 ? p->summed : nullptr, N, keep, p->cfg.Hkv, p->cfg.batch, p->status);
    p->launches += 1;
    IPOT_CUDA(cudaGetLastError());
    if (ev) IPOT_CUDA(cudaEventRecord(ev[3], p->stream));

    const int row_vecs = p->row_bytes / 16;
    const int slices = p->compact_slices;
    const size_t unit_vecs = (size_t)p->cfg.pot_size * row_vecs;
    if (!p->rope) {
        // programmatic dependent launch: the grid is set up while the selection still runs and waits inside the kernel
        cudaLaunchConfig_t lc = {};
        lc.gridDim = dim3(slices, 2, p->units);
        lc.blockDim = dim3(kMoveThreads, 1, 1);
        lc.stream = p->stream;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = at;
        lc.numAttrs = 1;
        IPOT_CUDA(cudaLaunchKernelEx(&lc, compact_kernel, (uint4 *)p->K, (uint4 *)p->V, (const int32_t *)p->idx, keep, N, row_vecs,
                                     row_vecs / slices, unit_vecs, p->status, pending_rows(p)));
        p->launches += 1;
    } else {
        launch_compact_rope(p, keep, N, row_vecs, unit_vecs);
        p->launches += 1;
    }
    IPOT_CUDA(cudaGetLastError());
    p->pend_K = p->pend_V = nullptr;  // the survivors are in the pot, the rest of the chunk is dropped
    if (ev) {
        IPOT_CUDA(cudaEventRecord(ev[4], p->stream));
        p->ev_used += 1;
    }
    p->len = keep;
    return IPOT_OK;
}

}  // namespace

namespace {
template <typename T>
int launch_novelty(ipot *p, const void *logits, size_t row_stride, const int32_t *labels, int n_tokens, int vocab,
                   float *out, size_t out_stride, int slot0)
{
    const size_t rows = (size_t)p->cfg.batch * n_tokens;
    const int segs = (vocab + kNovSegElems - 1) / kNovSegElems;
    int *counters = reinterpret_cast<int *>(p->nov_scratch);
    float2 *partial = reinterpret_cast<float2 *>(p->nov_scratch + kNovCounterBytes);
    dim3 grid(segs, (unsigned)rows);
    novelty_kernel<T><<<grid, kNovThreads, 0, p->stream>>>((const T *)logits, row_stride, vocab, segs, partial, counters, labels,
                                                           n_tokens, out, out_stride, slot0, p->status);
    p->launches += 1;
    IPOT_CUDA(cudaGetLastError());
    return IPOT_OK;
}
}  // namespace

// Blocks of one decode launch are equally long, so they run in waves over the resident slots, and every block
// pays a start-up and a merge.  Measured on 64 to 256 units: the fewest splits per unit whose last wave is at
// least 85 % full win (256 blocks on 296 slots beat 384, 768 or 2048); if no count up to 32 gets there, the fullest.
int decode_splits(int units, int slots)
{
    int best = 1;
    double best_eff = 0.0;
    for (int s = 1; s <= 32; ++s) {
        const double waves = (double)units * s / slots;
        const double eff = waves / std::ceil(waves);
        if (eff >= 0.85) return s;
        if (eff > best_eff + 1e-9) {
            best_eff = eff;
            best = s;
        }
    }
    return best;
}

template <typename T, int G>
int launch_decode_g(ipot *p, const void *q, float *out, float *lse)
{
    const int d = p->cfg.d, N = p->len;
    int splits = p->dec_splits;
    const int tile_keys = kDecStageVecs / (p->row_bytes / 16);
    if (splits > (N + tile_keys - 1) / tile_keys) splits = (N + tile_keys - 1) / tile_keys;  // at least one stage of rows per block
    const size_t smem = decode_smem_bytes(G, d);
    auto kern = decode_attn_kernel<T, G>;
    if (smem > 48 * 1024) IPOT_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    dim3 grid(splits, p->units);
    kern<<<grid, kDecThreads, smem, p->stream>>>((const T *)score_keys(p), (const T *)p->V, (const T *)q, out, lse, p->dec_partial,
                                                 p->dec_counters, N, d, p->row_bytes / 16, (size_t)p->cfg.pot_size * d,
                                                 (float)(1.4426950408889634 / std::sqrt((double)d)));
    p->launches += 1;
    IPOT_CUDA(cudaGetLastError());
    return IPOT_OK;
}

// bf16 rows of 64 or 128 channels: the tensor-core stream
template <int D>
int launch_decode_mma(ipot *p, const void *q, float *out, float *lse)
{
    const int N = p->len;
    int splits = p->dec_splits;
    if (splits > (N + 63) / 64) splits = (N + 63) / 64;  // at least one 16-key tile per warp
    const size_t smem = decode_mma_smem_bytes(p->G, D);
    auto kern = decode_attn_mma_kernel<D>;
    IPOT_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    dim3 grid(splits, p->units);
    kern<<<grid, kMmaWarps * 32, smem, p->stream>>>((const __nv_bfloat16 *)score_keys(p), (const __nv_bfloat16 *)p->V,
                                                    (const __nv_bfloat16 *)q, out, lse, p->dec_partial, p->dec_counters, N, p->G,
                                                    (size_t)p->cfg.pot_size * D, (float)(1.4426950408889634 / std::sqrt((double)D)));
    p->launches += 1;
    IPOT_CUDA(cudaGetLastError());
    return IPOT_OK;
}

template <typename T>
int launch_decode(ipot *p, const void *q, float *out, float *lse)
{
    switch (p->G) {
    case 1: return launch_decode_g<T, 1>(p, q, out, lse);
    case 2: return launch_decode_g<T, 2>(p, q, out, lse);
    case 4: return launch_decode_g<T, 4>(p, q, out, lse);
    case 8: return launch_decode_g<T, 8>(p, q, out, lse);
    default: return IPOT_E_INVALID;
    }
}

extern "C" {

int ipot_create(int pot_size, int keep, int layers, int Hq, int Hkv, int d, ipot_t **out)
{
    ipot_config_t c;
    memset(&c, 0, sizeof(c));
    c.pot_size = pot_size; c.keep = keep; c.layers = layers; c.Hq = Hq; c.Hkv = Hkv; c.d = d;
    c.batch = 1; c.dtype = IPOT_BF16; c.nuc_slots = -1; c.max_cap_rows = 64; c.stream = nullptr;
    return ipot_create_ex(&c, out);
}

int ipot_create_ex(const ipot_config_t *cfg, ipot_t **out)
{
    if (!cfg || !out) return IPOT_E_INVALID;
    int rc = check_config(*cfg);
    if (rc != IPOT_OK) return rc;
    ipot *p = new (std::nothrow) ipot();
    if (!p) return IPOT_E_NOMEM;
    p->cfg = *cfg;
    if (p->cfg.nuc_slots < 0) p->cfg.nuc_slots = p->cfg.keep / 2;
    p->G = cfg->Hq / cfg->Hkv;
    p->units = cfg->layers * cfg->batch * cfg->Hkv;
    p->elem_bytes = cfg->dtype == IPOT_F32 ? 4 : 2;
    p->row_bytes = cfg->d * p->elem_bytes;
    p->stream = (cudaStream_t)cfg->stream;
    p->scorer = IPOT_SCORER_AUTO;
    if (cudaGetDevice(&p->device) != cudaSuccess ||
        cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device) != cudaSuccess) {
        cudaGetLastError();
        delete p;
        return IPOT_E_CUDA;
    }
    const size_t pot_bytes = (size_t)p->units * cfg->pot_size * p->row_bytes;
    const int maxM = p->G * cfg->max_cap_rows;
    p->max_parts = (maxM + 127) / 128;
    const size_t score_elems = (size_t)p->units * cfg->pot_size;
    bool ok = true;
    auto alloc = [&](void **ptr, size_t bytes) {
        if (ok && cudaMalloc(ptr, bytes ? bytes : 16) != cudaSuccess) ok = false;
    };
    alloc(&p->K, pot_bytes);
    alloc(&p->V, pot_bytes);
    alloc((void **)&p->scores, score_elems * 4 * p->max_parts);
    alloc((void **)&p->summed, score_elems * 4);
    alloc((void **)&p->row_stats, (size_t)p->units * maxM * sizeof(float2));
    alloc((void **)&p->cap_stats, (size_t)p->units * maxM * sizeof(float2));
    alloc((void **)&p->mma_part, (size_t)kMmaSplits * p->units * maxM * sizeof(float2));
    alloc((void **)&p->nuc_mask, (size_t)cfg->batch * cfg->pot_size);
    alloc((void **)&p->idx, (size_t)p->units * cfg->keep * 4);
    alloc((void **)&p->status, 16);
    p->dec_splits = decode_splits(p->units, 2 * p->sm_count);  // both decode kernels keep two blocks per SM
    alloc((void **)&p->dec_partial, (size_t)p->units * p->dec_splits * p->G * (cfg->d + 2) * sizeof(float));
    alloc((void **)&p->dec_counters, (size_t)p->units * sizeof(int));
    alloc(&p->stage_q, (size_t)p->units * maxM * p->row_bytes);
    alloc(&p->stage_kc, (size_t)p->units * cfg->max_cap_rows * p->row_bytes);
    alloc((void **)&p->stage_aux, (size_t)cfg->batch * cfg->pot_size * 4);
    if (ok) ok = cudaMemset(p->status, 0, 16) == cudaSuccess && cudaMemset(p->dec_counters, 0, (size_t)p->units * sizeof(int)) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        free_all(p);
        delete p;
        return IPOT_E_NOMEM;
    }
    // kernels whose dynamic shared memory can exceed the default limit
    ok = cudaFuncSetAttribute(cap_row_stats<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)simt_smem_bytes(256)) == cudaSuccess &&
         cudaFuncSetAttribute(cap_column_sums<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)simt_smem_bytes(256)) == cudaSuccess &&
         cudaFuncSetAttribute(cap_row_stats<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)simt_smem_bytes(256)) == cudaSuccess &&
         cudaFuncSetAttribute(cap_column_sums<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)simt_smem_bytes(256)) == cudaSuccess &&
         cudaFuncSetAttribute(cap_self_stats_bf16, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)self_smem_bytes(256)) == cudaSuccess &&
         cudaFuncSetAttribute(cap_row_stats_mma, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)mma_scorer_smem_bytes(256)) == cudaSuccess &&
         cudaFuncSetAttribute(cap_column_sums_mma, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)mma_scorer_smem_bytes(256)) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        free_all(p);
        delete p;
        return IPOT_E_CUDA;
    }
    if (cudaStreamCreateWithFlags(&p->side, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&p->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&p->ev_join, cudaEventDisableTiming) != cudaSuccess) {
        cudaGetLastError();
        free_all(p);
        delete p;
        return IPOT_E_CUDA;
    }
    p->compact_slices = compact_slices(p);
    p->rope_slices = rope_slices(p);
    tc_plan_init(p->tc, p->cfg, p->K, p->sm_count);
    *out = p;
    return IPOT_OK;
}

int ipot_destroy(ipot_t *p)
{
    if (!p) return IPOT_OK;
    cudaStreamSynchronize(p->stream);
    free_all(p);
    delete p;
    return IPOT_OK;
}

int ipot_set_stream(ipot_t *p, void *s)
{
    if (!p) return IPOT_E_INVALID;
    int rc = materialise(p, true, true);  // queued on the stream that is being left
    if (rc != IPOT_OK) return rc;
    p->stream = (cudaStream_t)s;
    return IPOT_OK;
}

int ipot_set_nuc_slots(ipot_t *p, int T)
{
    if (!p || T < 0 || T > p->cfg.keep) return IPOT_E_INVALID;
    p->cfg.nuc_slots = T;
    return IPOT_OK;
}

int ipot_set_scorer(ipot_t *p, int scorer)
{
    if (!p || scorer < IPOT_SCORER_AUTO || scorer > IPOT_SCORER_TENSOR_SWEEPS) return IPOT_E_INVALID;
    p->scorer = scorer;
    return IPOT_OK;
}

int ipot_set_tuning(ipot_t *p, int what, long long value)
{
    if (!p) return IPOT_E_INVALID;
    switch (what) {
    case IPOT_TUNE_SWEEPS_CLUSTER:
        if (value != 0 && value != 1 && value != 2 && value != 4 && value != 8) return IPOT_E_INVALID;
        p->ts.cluster = (int)value;
        return IPOT_OK;
    case IPOT_TUNE_SWEEPS_FMA_EIGHTHS:
        if (value != -1 && value != 2 && value != 3) return IPOT_E_INVALID;
        p->ts.poly = (int)value;
        return IPOT_OK;
    case IPOT_TUNE_WAIT_LIMIT_NS:
        if (value < 1000) return IPOT_E_INVALID;
        p->ts.wait_ns = (unsigned long long)value;
        return IPOT_OK;
    case IPOT_TUNE_TEST_WITHHOLD_RANK:
        if (value < -1 || value > 7) return IPOT_E_INVALID;
        p->ts.withhold_rank = (int)value;
        return IPOT_OK;
    default:
        return IPOT_E_INVALID;
    }
}

int ipot_set_deferred_append(ipot_t *p, int on)
{
    if (!p) return IPOT_E_INVALID;
    if (!on) {
        int rc = materialise(p, true, true);
        if (rc != IPOT_OK) return rc;
    }
    p->deferred = on ? 1 : 0;
    return IPOT_OK;
}

int ipot_reset(ipot_t *p)
{
    if (!p) return IPOT_E_INVALID;
    p->len = 0;
    p->pend_K = p->pend_V = nullptr;
    p->tc.last_items = 0;  // the tensor scorer clears its statistics array before its next launch
    return IPOT_OK;
}

int ipot_append_chunk(ipot_t *p, const void *K, const void *V, int n)
{
    if (!p || !K || !V || n <= 0 || !aligned16(K) || !aligned16(V)) return IPOT_E_INVALID;
    if (p->len + n > p->cfg.pot_size) return IPOT_E_STATE;
    const size_t row_vecs = p->row_bytes / 16;
    const size_t n_vecs = (size_t)n * row_vecs;
    int pieces = (int)((n_vecs + (size_t)kMoveThreads * kMoveVecs - 1) / ((size_t)kMoveThreads * kMoveVecs));
    if (pieces < 1) pieces = 1;
    int rc = materialise(p, true, true);  // at most one chunk is kept outside the pot
    if (rc != IPOT_OK) return rc;
    if (p->deferred) {
        p->pend_first = p->len;
        p->pend_n = n;
        p->pend_V = V;
        if (!p->rope) {
            p->pend_K = K;
        } else {  // the rotated copy is what the scorers read: the keys go into the pot now, the values wait
            launch_append_rope(p, K, n_vecs, nullptr, n);
            p->launches += 1;
            IPOT_CUDA(cudaGetLastError());
        }
        p->len += n;
        return IPOT_OK;
    }
    if (!p->rope) {
        dim3 grid(pieces, p->units, 2);
        append_kernel<<<grid, kMoveThreads, 0, p->stream>>>((const uint4 *)K, (const uint4 *)V, (uint4 *)p->K, (uint4 *)p->V,
                                                           n_vecs, (size_t)p->cfg.pot_size * row_vecs, (size_t)p->len * row_vecs);
    } else {
        launch_append_rope(p, K, n_vecs, V, n);
    }
    p->launches += 1;
    IPOT_CUDA(cudaGetLastError());
    p->len += n;
    return IPOT_OK;
}

int ipot_append_chunk_host(ipot_t *p, const void *K, const void *V, int n)
{
    if (!p || !K || !V || n <= 0) return IPOT_E_INVALID;
    if (p->len + n > p->cfg.pot_size) return IPOT_E_STATE;
    int rc = materialise(p, true, true);
    if (rc != IPOT_OK) return rc;
    const size_t width = (size_t)n * p->row_bytes, dpitch = (size_t)p->cfg.pot_size * p->row_bytes;
    char *dK = (char *)p->K + (size_t)p->len * p->row_bytes, *dV = (char *)p->V + (size_t)p->len * p->row_bytes;
    IPOT_CUDA(cudaMemcpy2DAsync(dK, dpitch, K, width, width, p->units, cudaMemcpyHostToDevice, p->stream));
    IPOT_CUDA(cudaMemcpy2DAsync(dV, dpitch, V, width, width, p->units, cudaMemcpyHostToDevice, p->stream));
    if (p->rope) {  // the key rows are in place: rotate them into the copy
        launch_append_rope(p, dK, (size_t)p->cfg.pot_size * (p->row_bytes / 16), nullptr, n);
        p->launches += 1;
        IPOT_CUDA(cudaGetLastError());
    }
    p->len += n;
    return IPOT_OK;
}

int ipot_score_and_compress(ipot_t *p, const void *Q, int cap_rows, const float *aux)
{
    int rc = check_cycle_args(p, Q, cap_rows, aux, true);
    if (rc != IPOT_OK) return rc;
    if (!aligned16(Q) || (aux && (reinterpret_cast<uintptr_t>(aux) & 3u))) return IPOT_E_INVALID;
    return run_cycle(p, Q, nullptr, cap_rows, aux);
}

int ipot_score_and_compress_host(ipot_t *p, const void *Q, int cap_rows, const float *aux, int32_t *idx_host)
{
    int rc = check_cycle_args(p, Q, cap_rows, aux, true);
    if (rc != IPOT_OK) return rc;
    const size_t qbytes = (size_t)p->units * p->G * cap_rows * p->row_bytes;
    IPOT_CUDA(cudaMemcpyAsync(p->stage_q, Q, qbytes, cudaMemcpyHostToDevice, p->stream));
    if (aux) IPOT_CUDA(cudaMemcpyAsync(p->stage_aux, aux, (size_t)p->cfg.batch * p->len * 4, cudaMemcpyHostToDevice, p->stream));
    rc = run_cycle(p, p->stage_q, nullptr, cap_rows, aux ? p->stage_aux : nullptr);
    if (rc != IPOT_OK) return rc;
    if (idx_host)
        IPOT_CUDA(cudaMemcpyAsync(idx_host, p->idx, (size_t)p->units * p->cfg.keep * 4, cudaMemcpyDeviceToHost, p->stream));
    return IPOT_OK;
}

namespace {
int score_only(ipot *p, const void *Q, const void *Kc, int cap_rows, const float *aux)
{
    int parts = 1;
    int rc = run_scoring(p, Q, Kc, cap_rows, aux, &parts);
    if (rc != IPOT_OK) return rc;
    if (parts > 1) {
        const size_t n = (size_t)p->units * p->len;
        sum_parts_kernel<<<(unsigned)((n + 255) / 256), 256, 0, p->stream>>>(
            p->scores, parts, (size_t)p->units * p->cfg.pot_size, p->summed, n);
        p->launches += 1;
        IPOT_CUDA(cudaGetLastError());
    }
    return IPOT_OK;
}
}  // namespace

int ipot_score_only(ipot_t *p, const void *Q, int cap_rows, const float *aux)
{
    int rc = check_cycle_args(p, Q, cap_rows, aux, false);
    if (rc != IPOT_OK) return rc;
    if (!aligned16(Q)) return IPOT_E_INVALID;
    return score_only(p, Q, nullptr, cap_rows, aux);
}

int ipot_score_and_compress_cap(ipot_t *p, const void *Q, const void *K_cap, int cap_rows, const float *aux)
{
    int rc = check_cycle_args(p, Q, cap_rows, aux, true);
    if (rc != IPOT_OK) return rc;
    if (!K_cap || !aligned16(Q) || !aligned16(K_cap) || (aux && (reinterpret_cast<uintptr_t>(aux) & 3u))) return IPOT_E_INVALID;
    return run_cycle(p, Q, K_cap, cap_rows, aux);
}

int ipot_score_and_compress_cap_host(ipot_t *p, const void *Q, const void *K_cap, int cap_rows, const float *aux, int32_t *idx_host)
{
    int rc = check_cycle_args(p, Q, cap_rows, aux, true);
    if (rc != IPOT_OK) return rc;
    if (!K_cap) return IPOT_E_INVALID;
    const size_t qbytes = (size_t)p->units * p->G * cap_rows * p->row_bytes, kcbytes = (size_t)p->units * cap_rows * p->row_bytes;
    IPOT_CUDA(cudaMemcpyAsync(p->stage_q, Q, qbytes, cudaMemcpyHostToDevice, p->stream));
    IPOT_CUDA(cudaMemcpyAsync(p->stage_kc, K_cap, kcbytes, cudaMemcpyHostToDevice, p->stream));
    if (aux) IPOT_CUDA(cudaMemcpyAsync(p->stage_aux, aux, (size_t)p->cfg.batch * p->len * 4, cudaMemcpyHostToDevice, p->stream));
    rc = run_cycle(p, p->stage_q, p->stage_kc, cap_rows, aux ? p->stage_aux : nullptr);
    if (rc != IPOT_OK) return rc;
    if (idx_host)
        IPOT_CUDA(cudaMemcpyAsync(idx_host, p->idx, (size_t)p->units * p->cfg.keep * 4, cudaMemcpyDeviceToHost, p->stream));
    return IPOT_OK;
}

int ipot_score_only_cap(ipot_t *p, const void *Q, const void *K_cap, int cap_rows, const float *aux)
{
    int rc = check_cycle_args(p, Q, cap_rows, aux, false);
    if (rc != IPOT_OK) return rc;
    if (!K_cap || !aligned16(Q) || !aligned16(K_cap)) return IPOT_E_INVALID;
    return score_only(p, Q, K_cap, cap_rows, aux);
}

int ipot_nuc_scores(ipot_t *p, const void *logits, int logits_dtype, long long row_stride, const int32_t *labels,
                    int n_tokens, int vocab, float *aux_out, long long aux_stride, int slot0)
{
    if (!p || !logits || !labels || !aux_out) return IPOT_E_INVALID;
    if (logits_dtype != IPOT_BF16 && logits_dtype != IPOT_F32) return IPOT_E_INVALID;
    if (n_tokens < 1 || n_tokens > kNovMaxRows / p->cfg.batch || vocab < 1 || row_stride < vocab) return IPOT_E_INVALID;
    if (slot0 < 0 || aux_stride < (long long)slot0 + n_tokens) return IPOT_E_INVALID;
    const size_t elem = logits_dtype == IPOT_F32 ? 4 : 2;
    if ((reinterpret_cast<uintptr_t>(logits) % elem) || (reinterpret_cast<uintptr_t>(labels) & 3u) ||
        (reinterpret_cast<uintptr_t>(aux_out) & 3u))
        return IPOT_E_INVALID;
    const size_t rows = (size_t)p->cfg.batch * n_tokens;
    const size_t need = rows * ((vocab + kNovSegElems - 1) / kNovSegElems);
    if (!p->nov_scratch || need > p->nov_capacity) {  // first use or a larger shape: the only allocation outside ipot_create
        IPOT_CUDA(cudaStreamSynchronize(p->stream));
        cudaFree(p->nov_scratch);  // only this call's own scratch: every other buffer keeps its owner
        p->nov_scratch = nullptr;
        p->nov_capacity = 0;
        if (cudaMalloc((void **)&p->nov_scratch, kNovCounterBytes + need * sizeof(float2)) != cudaSuccess) {
            cudaGetLastError();
            return IPOT_E_NOMEM;
        }
        IPOT_CUDA(cudaMemsetAsync(p->nov_scratch, 0, kNovCounterBytes, p->stream));
        p->nov_capacity = need;
    }
    return logits_dtype == IPOT_F32
               ? launch_novelty<float>(p, logits, (size_t)row_stride, labels, n_tokens, vocab, aux_out, (size_t)aux_stride, slot0)
               : launch_novelty<__nv_bfloat16>(p, logits, (size_t)row_stride, labels, n_tokens, vocab, aux_out, (size_t)aux_stride, slot0);
}

int ipot_decode_attention(ipot_t *p, const void *q, float *out, float *lse)
{
    if (!p || !q || !out || !aligned16(q) || (reinterpret_cast<uintptr_t>(out) & 3u) || (reinterpret_cast<uintptr_t>(lse) & 3u))
        return IPOT_E_INVALID;
    const int lpk = p->row_bytes / 16;
    if (p->row_bytes % 16 || (lpk != 4 && lpk != 8 && lpk != 16 && lpk != 32)) return IPOT_E_INVALID;
    if (p->G > 8) return IPOT_E_INVALID;
    if (p->len < 1) return IPOT_E_STATE;
    int rc = materialise(p, true, true);
    if (rc != IPOT_OK) return rc;
    if (p->cfg.dtype == IPOT_BF16 && p->scorer != IPOT_SCORER_SIMT && (p->cfg.d == 64 || p->cfg.d == 128))
        return p->cfg.d == 64 ? launch_decode_mma<64>(p, q, out, lse) : launch_decode_mma<128>(p, q, out, lse);
    if (p->G != 1 && p->G != 2 && p->G != 4 && p->G != 8) return IPOT_E_INVALID;
    return p->cfg.dtype == IPOT_F32 ? launch_decode<float>(p, q, out, lse) : launch_decode<__nv_bfloat16>(p, q, out, lse);
}

int ipot_enable_rope(ipot_t *p, const void *cos_table, const void *sin_table, int pairing)
{
    if (!p || !cos_table || !sin_table || !aligned16(cos_table) || !aligned16(sin_table)) return IPOT_E_INVALID;
    if (pairing != IPOT_ROPE_HALF && pairing != IPOT_ROPE_INTERLEAVED) return IPOT_E_INVALID;
    if (p->row_bytes % 32) return IPOT_E_INVALID;  // a row must split into two halves of whole 16-byte vectors
    if (p->len != 0) return IPOT_E_STATE;
    if (!p->Krot) {
        IPOT_CUDA(cudaStreamSynchronize(p->stream));
        if (cudaMalloc(&p->Krot, (size_t)p->units * p->cfg.pot_size * p->row_bytes) != cudaSuccess) {
            cudaGetLastError();
            p->Krot = nullptr;
            return IPOT_E_NOMEM;
        }
    }
    p->rope_cos = cos_table;
    p->rope_sin = sin_table;
    p->rope = pairing;
    return IPOT_OK;
}

int ipot_view_rope(ipot_t *p, void **K_rot)
{
    if (!p || !K_rot) return IPOT_E_INVALID;
    if (!p->rope) return IPOT_E_STATE;
    *K_rot = p->Krot;
    return IPOT_OK;
}

int ipot_view(ipot_t *p, void **K, void **V, int *len)
{
    if (!p) return IPOT_E_INVALID;
    int rc = materialise(p, true, true);
    if (rc != IPOT_OK) return rc;
    if (K) *K = p->K;
    if (V) *V = p->V;
    if (len) *len = p->len;
    return IPOT_OK;
}

int ipot_last_indices(ipot_t *p, const int32_t **idx)
{
    if (!p || !idx) return IPOT_E_INVALID;
    *idx = p->idx;
    return IPOT_OK;
}

int ipot_last_scores(ipot_t *p, const float **u, int *len_before)
{
    if (!p || !u) return IPOT_E_INVALID;
    *u = p->last_scores ? p->last_scores : p->scores;
    if (len_before) *len_before = p->last_len_before;
    return IPOT_OK;
}

int ipot_sync_status(ipot_t *p)
{
    if (!p) return IPOT_E_INVALID;
    int rc = materialise(p, true, true);  // after this call the caller's chunk buffers are free again
    if (rc != IPOT_OK) return rc;
    IPOT_CUDA(cudaStreamSynchronize(p->stream));
    int st = 0;
    IPOT_CUDA(cudaMemcpy(&st, p->status, sizeof(int), cudaMemcpyDeviceToHost));
    return st;
}

int ipot_set_profiling(ipot_t *p, int on)
{
    if (!p) return IPOT_E_INVALID;
    if (on && !p->ev) {  // the event pool is created on first use
        p->ev = new (std::nothrow) cudaEvent_t[kProfSlots][5]();
        if (!p->ev) return IPOT_E_NOMEM;
        for (int i = 0; i < kProfSlots; ++i)
            for (auto &e : p->ev[i]) IPOT_CUDA(cudaEventCreate(&e));
    }
    p->profiling = on != 0;
    p->ev_used = 0;
    return IPOT_OK;
}

int ipot_kernel_ms(ipot_t *p, float ms[4], int *cycles, int *scorer_used)
{
    if (!p || !ms) return IPOT_E_INVALID;
    if (!p->profiling || p->ev_used == 0) return IPOT_E_STATE;
    IPOT_CUDA(cudaEventSynchronize(p->ev[p->ev_used - 1][4]));
    double sum[4] = {0, 0, 0, 0};
    for (int c = 0; c < p->ev_used; ++c)
        for (int i = 0; i < 4; ++i) {
            float t = 0.f;
            IPOT_CUDA(cudaEventElapsedTime(&t, p->ev[c][i], p->ev[c][i + 1]));
            sum[i] += t;
        }
    for (int i = 0; i < 4; ++i) ms[i] = (float)(sum[i] / p->ev_used);
    if (cycles) *cycles = p->ev_used;
    if (scorer_used) *scorer_used = p->last_scorer;
    p->ev_used = 0;
    return IPOT_OK;
}

int ipot_launch_count(ipot_t *p, long long *launches)
{
    if (!p || !launches) return IPOT_E_INVALID;
    *launches = p->launches;
    return IPOT_OK;
}

const char *ipot_strerror(int code)
{
    switch (code) {
    case IPOT_OK: return "ok";
    case IPOT_E_INVALID: return "invalid argument";
    case IPOT_E_STATE: return "call not allowed in the pot's current state";
    case IPOT_E_NOMEM: return "out of memory";
    case IPOT_E_CUDA: return "CUDA call failed or no usable device";
    case IPOT_E_TIMEOUT: return "a bounded device-side wait gave up";
    case IPOT_E_BOUNDS: return "a device-side self-check found an index out of range";
    case IPOT_E_LIMIT: return "size exceeds the fixed scratch capacity of the allocation-free entry point";
    default: return "unknown error code";
    }
}

}  // extern "C"

// ---------------------------------------------------------------------------
// Allocation-free CaP scoring.  The two SIMT launches hand the per-row softmax
// statistics to each other through global memory; here that scratch is a fixed
// array inside the library image instead of a cudaMalloc'ed buffer.
// ---------------------------------------------------------------------------
static __device__ __align__(256) float2 g_noalloc_row_stats[IPOT_NOALLOC_MAX_ROWS];

namespace {
std::mutex g_noalloc_mutex;
float2 *g_noalloc_ptr[64];  // device address of the array, per device ordinal

// The array's name is only a host-side handle; kernels need the address the
// runtime reports for the device that is current.
int noalloc_scratch(float2 **out)
{
    int dev = 0;
    IPOT_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return IPOT_E_INVALID;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
        void *ptr = nullptr;
        IPOT_CUDA(cudaGetSymbolAddress(&ptr, g_noalloc_row_stats));
        g_noalloc_ptr[dev] = static_cast<float2 *>(ptr);
    }
    *out = g_noalloc_ptr[dev];
    return IPOT_OK;
}

template <typename T>
int noalloc_launch(const void *Q, const void *K, float *scores, float2 *stats, int units, int M, int N, int d,
                   size_t k_unit_rows, cudaStream_t stream)
{
    const size_t smem = simt_smem_bytes(d);
    IPOT_CUDA(cudaFuncSetAttribute(cap_row_stats<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)simt_smem_bytes(256)));
    IPOT_CUDA(cudaFuncSetAttribute(cap_column_sums<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)simt_smem_bytes(256)));
    const float scale_log2e = (float)(1.4426950408889634 / std::sqrt((double)d));
    dim3 g1((M + kSimtRows - 1) / kSimtRows, units), g2((N + kSimtKeys - 1) / kSimtKeys, units);
    cap_row_stats<T><<<g1, kSimtThreads, smem, stream>>>((const T *)Q, (const T *)K, stats, M, N, d, k_unit_rows * d, scale_log2e, nullptr, 0, 1);
    cap_column_sums<T><<<g2, kSimtThreads, smem, stream>>>((const T *)Q, (const T *)K, stats, scores, M, N, d, k_unit_rows * d, scale_log2e);
    IPOT_CUDA(cudaGetLastError());
    return IPOT_OK;
}
}  // namespace

extern "C" int ipot_cap_scores_noalloc(const void *Q, const void *K, float *scores, int units, int rows, int N, int d,
                                       int k_unit_rows, int dtype, void *cuda_stream)
{
    if (!Q || !K || !scores || !aligned16(Q) || !aligned16(K) || (reinterpret_cast<uintptr_t>(scores) & 3u))
        return IPOT_E_INVALID;
    if (units < 1 || rows < 1 || N < 1 || k_unit_rows < N || d < 32 || d > 256 || d % 8) return IPOT_E_INVALID;
    if (dtype != IPOT_BF16 && dtype != IPOT_F32) return IPOT_E_INVALID;
    if ((long long)units * rows > IPOT_NOALLOC_MAX_ROWS) return IPOT_E_LIMIT;
    float2 *stats = nullptr;
    int rc = noalloc_scratch(&stats);
    if (rc != IPOT_OK) return rc;
    // every statistics entry that the second launch reads is written by the first one,
    // so nothing left behind by an earlier call needs clearing
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    return dtype == IPOT_F32
               ? noalloc_launch<float>(Q, K, scores, stats, units, rows, N, d, (size_t)k_unit_rows, stream)
               : noalloc_launch<__nv_bfloat16>(Q, K, scores, stats, units, rows, N, d, (size_t)k_unit_rows, stream);
}
