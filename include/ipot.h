/*
 * ipot.h - C ABI of the memory-pot library: the Continual Context Distillation
 * (CCD) compression cycle of InfiniPot (arxiv 2410.01518) on one CUDA device.
 *
 * The pot is the paper's fixed-size KV cache (Sec. 3.1: at most |M| entries;
 * Sec. 3.2: filled sequentially, then distilled to |C| entries, then filled
 * again).  One pot object holds, for every (layer, stream, kv-head) "unit", a
 * K and a V array of pot_size rows of d elements.
 *
 * Memory layouts (all dense, row-major, innermost index last):
 *   pot K, V     [layers][batch][Hkv][pot_size][d]   element = bf16 or f32
 *   chunk K, V   [layers][batch][Hkv][n_tokens][d]   same element type
 *   Q_cap        [layers][batch][Hq][cap_rows][d]    same element type
 *   aux_scores   [batch][len]                        f32, higher = more novel
 *   scores       [layers][batch][Hkv][len]           f32
 *   indices      [layers][batch][Hkv][keep]          int32, strictly ascending
 * Query head h attends to KV head h / (Hq / Hkv).
 *
 * Conventions
 *   - Every function returns IPOT_OK (0) or a negative IPOT_E_* code; nothing
 *     is thrown across the boundary.  ipot_strerror() names a code.
 *   - Argument and state errors are found on the host before anything is
 *     launched and leave the pot unchanged.
 *   - Unless a function's name ends in _host, its data pointers are DEVICE
 *     pointers on the pot's device, 16-byte aligned, owned by the caller and
 *     only read.  Work is queued on the pot's stream and the call returns
 *     without waiting; the caller must keep the buffers alive and unchanged
 *     until that work has run (synchronise the stream or call
 *     ipot_sync_status()).  Inside a cycle the library may run a kernel on a
 *     stream of its own beside the others; it is forked from and joined back
 *     into the pot's stream by events within the same call, so everything a
 *     call has queued is ordered in the pot's stream when the call returns.
 *   - The library owns the pot, the score/index arrays and its scratch; they
 *     are allocated in ipot_create*() and freed in ipot_destroy().
 *   - A pot object is not thread-safe; use one host thread per pot at a time.
 *   - There is no CPU fallback: without a usable CUDA device every call that
 *     touches data fails with IPOT_E_CUDA.
 */
#ifndef IPOT_H
#define IPOT_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ipot ipot_t; /* opaque, library-owned */

enum {
    IPOT_OK = 0,
    IPOT_E_INVALID = -1, /* bad argument (NULL, misaligned, out of range, unsupported shape) */
    IPOT_E_STATE = -2,   /* call not allowed in the pot's current state (overflow, nothing to distil) */
    IPOT_E_NOMEM = -3,   /* device or host allocation failed */
    IPOT_E_CUDA = -4,    /* a CUDA runtime/driver call failed, or no device */
    IPOT_E_TIMEOUT = -5, /* a bounded device-side wait gave up (sticky, reported by ipot_sync_status) */
    IPOT_E_BOUNDS = -6,  /* a device-side self-check found an index out of range (sticky) */
    IPOT_E_LIMIT = -7    /* a size exceeds the fixed scratch of ipot_cap_scores_noalloc() */
};

enum { IPOT_BF16 = 0, IPOT_F32 = 1 };

/* Channel pairing of the rotary embedding (ipot_enable_rope). */
enum {
    IPOT_ROPE_HALF = 1,        /* channel c with c + d/2 */
    IPOT_ROPE_INTERLEAVED = 2  /* channel 2c with 2c + 1 */
};

/* Which scoring kernel ipot_score_and_compress() uses. */
enum {
    IPOT_SCORER_AUTO = 0,   /* the fastest kernel the shape allows: tcgen05, else warp-level tensor cores, else fp32 FMAs */
    IPOT_SCORER_SIMT = 1,   /* fp32 FMA kernel: any supported shape, f32 or bf16 */
    IPOT_SCORER_TENSOR = 2, /* tcgen05 kernel (bf16, d = 64 or 128): IPOT_E_INVALID if the shape does not allow it */
    IPOT_SCORER_WARP_MMA = 3, /* warp-level tensor-core kernels (bf16, d a multiple of 16): what AUTO takes for bf16
                                pots the tcgen05 kernel does not; IPOT_E_INVALID if the shape does not allow it */
    IPOT_SCORER_TENSOR_SWEEPS = 4 /* tcgen05 kernel that goes over the keys twice (row log-sum-exps, then probabilities
                                and their column sums) inside thread-block clusters, so that no block waits for a block
                                it is not co-scheduled with (bf16, d = 64 or 128, at most 512 folded query rows):
                                IPOT_E_INVALID if the shape does not allow it */
};

typedef struct {
    int pot_size;     /* context slots per unit (the paper's |M| minus the CaP rows) */
    int keep;         /* |C|: entries that survive a cycle, 0 < keep < pot_size */
    int layers, Hq, Hkv, d;
    int batch;        /* independent streams, >= 1 */
    int dtype;        /* IPOT_BF16 or IPOT_F32 */
    int nuc_slots;    /* T of Sec. 3.3.3, 0 <= T <= keep; -1 = keep / 2 (the 50 % ratio of Sec. 4.4.2) */
    int max_cap_rows; /* largest cap_rows that will be passed (scratch is sized for it) */
    void *stream;     /* cudaStream_t, NULL = the default stream */
} ipot_config_t;

/*
 * Sec. 3.1-3.2: create an empty pot (len = 0) on the current CUDA device with
 * batch = 1, bf16 elements, T = keep / 2, up to 64 CaP rows, default stream.
 * Limits: Hq % Hkv == 0; d a multiple of 8 with 32 <= d <= 256; 0 < keep <
 * pot_size <= 32768.  *out is set only on success.  Errors: INVALID, NOMEM, CUDA.
 */
int ipot_create(int pot_size, int keep, int layers, int Hq, int Hkv, int d, ipot_t **out);

/* Same, with every parameter explicit. */
int ipot_create_ex(const ipot_config_t *cfg, ipot_t **out);

/* Waits for the pot's queued work, frees everything.  NULL is accepted. */
int ipot_destroy(ipot_t *pot);

/* Use another cudaStream_t for all later calls (the caller orders the hand-over). */
int ipot_set_stream(ipot_t *pot, void *cuda_stream);

/* Sec. 3.3.3 / Sec. 4.4.2: number of slots T given to the novelty ranking, 0 <= T <= keep. */
int ipot_set_nuc_slots(ipot_t *pot, int T);

/* IPOT_SCORER_*; a tensor-core scorer is refused at the next cycle if the shape does not allow it. */
int ipot_set_scorer(ipot_t *pot, int scorer);

/*
 * Launch parameters of the scoring kernels (Eq. 2 itself is not affected; results stay within the stated
 * tolerances for every setting).  `what`:
 *   IPOT_TUNE_SWEEPS_CLUSTER      CTAs per thread-block cluster of IPOT_SCORER_TENSOR_SWEEPS: 1, 2, 4, 8, or 0 = chosen
 *                                 from the shape (the default)
 *   IPOT_TUNE_SWEEPS_FMA_EIGHTHS  how many eighths of that kernel's exponentials are evaluated as a polynomial on the
 *                                 FMA pipe instead of the special-function unit: 2, 3, or -1 = default
 *   IPOT_TUNE_WAIT_LIMIT_NS       time after which a device-side wait of a tensor-core scorer gives up and the launch
 *                                 ends with IPOT_E_TIMEOUT in the status word (default 200 ms; at least 1000).
 *                                 IPOT_SCORER_TENSOR_SWEEPS counts it from the start of each wait, IPOT_SCORER_TENSOR
 *                                 from the start of each thread block (a launch of either takes well under 1 ms)
 *   IPOT_TUNE_TEST_WITHHOLD_RANK  for tests of the give-up path only: CTA `value` (0-7) of every cluster
 *                                 (IPOT_SCORER_TENSOR_SWEEPS) or of the grid (IPOT_SCORER_TENSOR) never reports its
 *                                 statistics, so every wait for them runs into the limit; -1 = off (default)
 * Errors: INVALID (unknown `what`, value out of range).  Takes effect at the next launch.
 */
enum {
    IPOT_TUNE_SWEEPS_CLUSTER = 1,
    IPOT_TUNE_SWEEPS_FMA_EIGHTHS = 2,
    IPOT_TUNE_WAIT_LIMIT_NS = 3,
    IPOT_TUNE_TEST_WITHHOLD_RANK = 4
};
int ipot_set_tuning(ipot_t *pot, int what, long long value);

/* Forget the contents: len = 0.  Nothing is launched.  Also the way back to a defined state after
 * ipot_sync_status() reported IPOT_E_TIMEOUT: the scorer's exchange buffers are cleared before their next use
 * (the sticky status itself stays). */
int ipot_reset(ipot_t *pot);

/*
 * Sec. 3.2 (the free part of the cache is filled in order): copy n_tokens
 * new rows of every unit behind the rows already in the pot; len += n_tokens.
 * K, V: device, [layers][batch][Hkv][n_tokens][d].
 * Errors: INVALID (NULL, misaligned, n_tokens <= 0), STATE (len + n_tokens >
 * pot_size; the pot is unchanged), CUDA.
 */
int ipot_append_chunk(ipot_t *pot, const void *K, const void *V, int n_tokens);

/*
 * Deferred append (off by default).  While it is on, ipot_append_chunk() copies nothing: it notes the caller's
 * buffers, and the rows are taken from there when they are needed -
 *   - the tensor-core scorer reads the new keys in place (when the fill before the append is a multiple of 256;
 *     otherwise, and for every other scorer, the keys are copied into the pot first);
 *   - the compaction of the next cycle (Appendix B, "KV-cache compression") fetches the surviving rows from the
 *     chunk, so rows that the cycle drops are never copied and survivors move once instead of twice;
 *   - every other call that reads or exposes the pot's rows (ipot_view, ipot_decode_attention, a further append,
 *     ipot_append_chunk_host, ipot_set_stream, ipot_sync_status, turning the mode off) first queues the plain copy.
 * In rotary mode only the values are deferred (the scorers read the rotated copy, which is written at append).
 * The pot's contents after any of these calls are the same as without the mode.  What changes is the lifetime of
 * the chunk buffers: they must stay alive and unchanged until the next ipot_score_and_compress*() has run on the
 * stream or ipot_sync_status() has returned - synchronising the stream right after the append is not enough.
 * Errors: INVALID (NULL pot), CUDA.
 */
int ipot_set_deferred_append(ipot_t *pot, int on);

/* Same with HOST buffers (pinned memory makes the copy asynchronous): the
 * rows go straight from host memory into the pot with strided copies. */
int ipot_append_chunk_host(ipot_t *pot, const void *K_host, const void *V_host, int n_tokens);

/*
 * One CCD cycle (Sec. 3.2) over all units, N = len rows in the pot:
 *   1. Sec. 3.3.3: per stream, the T slots with the largest aux_scores are
 *      reserved in every head (ties: lower slot first);
 *   2. Sec. 3.3.1, Eq. 2: per unit, u_j = sum over the G*cap_rows query rows of
 *      the unit's KV head of softmax_j(q . k_j / sqrt(d)), the softmax taken
 *      over the N pot keys; fp32 arithmetic, probabilities never stored;
 *   3. Sec. 3.3.3 / Appendix B: per unit, the keep - T non-reserved slots with
 *      the largest u_j join the reserved ones (ties: lower slot first);
 *   4. Appendix B: K and V rows of the survivors are moved, in place and in
 *      their original order, to rows 0 .. keep-1; len = keep.
 * Q_cap: device [layers][batch][Hq][cap_rows][d]; aux_scores: device
 * [batch][len] f32, may be NULL iff T == 0.  All inputs must be finite.
 * Errors: INVALID (NULL, misaligned, cap_rows < 1 or > max_cap_rows, scorer
 * not applicable), STATE (len <= keep: nothing to distil; pot unchanged), CUDA.
 */
int ipot_score_and_compress(ipot_t *pot, const void *Q_cap, int cap_rows, const float *aux_scores);

/*
 * Same with HOST buffers: Q_cap_host and aux_host are copied to library-owned
 * device staging first; if idx_host is not NULL the index lists
 * ([layers][batch][Hkv][keep] int32) are copied back into it.  All copies are
 * queued on the pot's stream; with pageable memory they block the caller.
 */
int ipot_score_and_compress_host(ipot_t *pot, const void *Q_cap_host, int cap_rows,
                                 const float *aux_host, int32_t *idx_host);

/* Steps 1-2 of the cycle only: fills the score array, leaves the pot and len
 * untouched (aux_scores may be NULL: step 1 is then skipped). */
int ipot_score_only(ipot_t *pot, const void *Q_cap, int cap_rows, const float *aux_scores);

/*
 * The cycle with the CaP's own keys inside the softmax, as the PyTorch-style
 * listing of Appendix B ("Calculate Attention Score") computes it: the CaP
 * queries attend to every key of the sequence, the CaP included, under the
 * causal mask, and the CaP columns are cut away before the rows are summed.
 * CaP row i (0-based, within its query head) therefore normalises over the len
 * pot keys and the CaP keys 0..i of its KV head; the scores of a unit then sum to
 * less than G * cap_rows.  Selection and compaction are unchanged.
 *   K_cap : device, [layers][batch][Hkv][cap_rows][d], pot dtype, 16-byte
 *           aligned, caller-owned, read-only; the keys of the same cap_rows
 *           positions the queries of Q_cap belong to.
 * Everything else as in ipot_score_and_compress / ipot_score_only; a NULL K_cap
 * is IPOT_E_INVALID (use the plain calls for the context-only softmax).
 */
int ipot_score_and_compress_cap(ipot_t *pot, const void *Q_cap, const void *K_cap, int cap_rows,
                                const float *aux_scores);
int ipot_score_only_cap(ipot_t *pot, const void *Q_cap, const void *K_cap, int cap_rows,
                        const float *aux_scores);
/* ipot_score_and_compress_cap with HOST buffers (Q_cap, K_cap, aux staged on the device first; index
 * lists copied back if idx_host is not NULL), as ipot_score_and_compress_host. */
int ipot_score_and_compress_cap_host(ipot_t *pot, const void *Q_cap_host, const void *K_cap_host, int cap_rows,
                                     const float *aux_host, int32_t *idx_host);

/*
 * Token novelty, the quantity the NuC criterion ranks (Sec. 3.3.2, Eq. 3): for every new token the
 * cross-entropy of the model's prediction, n = -log softmax(z)[x] = log sum_v exp(z_v) - z_x, from the
 * logits z of the position that predicted the token and the token id x that followed.  The result can
 * be written straight into the aux_scores array of the next ipot_score_and_compress call.
 *   logits       : device, [batch][n_tokens] rows of `vocab` values, `row_stride` elements apart
 *                  (row_stride >= vocab), of type logits_dtype (IPOT_BF16 or IPOT_F32; need not be the
 *                  pot's type); rows that start on a 16-byte boundary are read with 16-byte loads,
 *                  others element by element.  Caller-owned, read-only.
 *   labels       : device, [batch][n_tokens] int32 token ids; a negative id marks an ignored position
 *                  (novelty 0); an id >= vocab also gives 0 and raises the sticky status IPOT_E_BOUNDS.
 *   aux_out      : device fp32; token t of stream b goes to aux_out[b * aux_stride + slot0 + t], i.e.
 *                  slot0 is the pot fill before the chunk was appended; aux_stride >= slot0 + n_tokens.
 * batch * n_tokens <= 65535.  Asynchronous on the pot's stream.  Uses a library-owned scratch of
 * 256 KiB + 8 * batch * n_tokens * ceil(vocab / 8192) bytes that is allocated on first use and when a
 * call needs more (those calls synchronise the stream and may return IPOT_E_NOMEM); no other allocation.
 * Errors: INVALID (NULL, sizes, alignment of the element type), NOMEM, CUDA.
 */
int ipot_nuc_scores(ipot_t *pot, const void *logits, int logits_dtype, long long row_stride,
                    const int32_t *labels, int n_tokens, int vocab, float *aux_out, long long aux_stride,
                    int slot0);

/*
 * Generation over the pot.  After a cycle the heads of a layer hold different tokens (the CaP score is per
 * head, Sec. 3.3.1), so each (layer, stream, kv-head) unit is its own cache; Sec. 4.5 measures generation
 * at a fixed pot.  For one new token: query head h attends to rows [0, len) of the unit of KV head
 * h / (Hq / Hkv):  out_h = sum_j softmax_j(q_h . k_j / sqrt(d)) v_j.
 *   q   : device, [layers][batch][Hq][d], pot dtype, 16-byte aligned (in rotary mode: rotated at the new
 *         token's position by the caller; the keys read are then the rotated copy).  Caller-owned.
 *   out : device, [layers][batch][Hq][d] fp32, normalised.
 *   lse : device, [layers][batch][Hq] fp32, or NULL: log sum_j exp(q_h . k_j / sqrt(d)), with which a
 *         caller merges this result with attention over tokens that are not in the pot.
 * bf16 pots with d = 64 or 128 and Hq / Hkv <= 8 run on warp-level tensor cores (fp32 accumulation, the
 * softmax weights kept to 16 mantissa bits); every other supported shape, and every shape after
 * ipot_set_scorer(IPOT_SCORER_SIMT), uses fp32 FMAs, which needs Hq / Hkv in {1, 2, 4, 8} and rows of 64,
 * 128, 256 or 512 bytes.  Unsupported shapes: IPOT_E_INVALID.
 * Requires len >= 1 (IPOT_E_STATE).  Asynchronous on the pot's stream; the pot is not changed.
 */
int ipot_decode_attention(ipot_t *pot, const void *q, float *out, float *lse);

/*
 * Context-reset rotary embedding (Sec. 3.4): the pot keeps its keys WITHOUT rotary embedding and every
 * slot j carries position j, so positions run 0 .. len-1 again after each cycle.  With this mode on, the
 * K rows passed to ipot_append_chunk are unrotated keys; the library maintains beside them a copy in
 * which slot j is rotated at position j (ipot_view_rope): appended rows are rotated at the slots they
 * land in, and a cycle rotates every row it moves at its new slot, inside the same kernels that move
 * the rows, so no separate pass over the pot follows a cycle.  The CaP queries of
 * ipot_score_and_compress attend to the rotated copy (the caller rotates Q_cap at the CaP's positions
 * len .. len + cap_rows - 1); ipot_view keeps returning the unrotated keys.
 *   cos_table, sin_table : device, [pot_size][d / 2] in the pot's dtype, 16-byte aligned, caller-owned
 *                          and read by every later append and cycle until ipot_destroy: cos and sin of
 *                          position x frequency (the paper fixes no base or scaling; they are the
 *                          model's).
 *   pairing              : IPOT_ROPE_HALF (channel c with c + d/2) or IPOT_ROPE_INTERLEAVED (2c, 2c + 1).
 * The rotation is evaluated in single precision as lo' = fma(lo, cos, -(hi * sin)),
 * hi' = fma(hi, cos, lo * sin) and rounded once to the pot's dtype.
 * Allowed only while the pot is empty (len == 0; else IPOT_E_STATE); needs d * element size to be a
 * multiple of 32 bytes (IPOT_E_INVALID otherwise).  The first call allocates the copy (pot_size rows per
 * unit; synchronises the stream; IPOT_E_NOMEM).  The mode stays on for the life of the pot.
 */
int ipot_enable_rope(ipot_t *pot, const void *cos_table, const void *sin_table, int pairing);

/* Borrowed device pointer to the rotated copy of the keys, [layers][batch][Hkv][pot_size][d]; rows >= len
 * are undefined.  IPOT_E_STATE unless ipot_enable_rope was called. */
int ipot_view_rope(ipot_t *pot, void **K_rot);

/*
 * Borrowed device pointers to the pot ([layers][batch][Hkv][pot_size][d]) and
 * the current fill.  Rows >= len are undefined.  The pointers stay valid until
 * ipot_destroy(); their contents are final once the stream's queued work ran.
 * Any of K, V, len may be NULL.
 */
int ipot_view(ipot_t *pot, void **K, void **V, int *len);

/* Results of the last cycle (device, library-owned, overwritten by the next cycle). */
int ipot_last_indices(ipot_t *pot, const int32_t **idx);            /* [layers][batch][Hkv][keep] */
int ipot_last_scores(ipot_t *pot, const float **u, int *len_before); /* [layers][batch][Hkv][len_before] */

/* Waits for the pot's stream and returns the sticky device status
 * (IPOT_OK, IPOT_E_TIMEOUT, IPOT_E_BOUNDS) or IPOT_E_CUDA. */
int ipot_sync_status(ipot_t *pot);

/*
 * Per-kernel device timing.  While enabled, every cycle (up to 2048 between
 * reads) records CUDA events on the pot's stream around its kernels; nothing
 * waits.  ipot_kernel_ms() waits for the last recorded cycle, returns the MEAN
 * over the recorded cycles in milliseconds - ms[0] NuC ranking, ms[1] CaP
 * scoring, ms[2] per-head selection, ms[3] K/V compaction - and starts a new
 * series.  *cycles (may be NULL) = cycles averaged; *scorer_used (may be NULL)
 * = IPOT_SCORER_SIMT, IPOT_SCORER_TENSOR or IPOT_SCORER_WARP_MMA.  STATE if nothing was recorded.
 */
int ipot_set_profiling(ipot_t *pot, int on);
int ipot_kernel_ms(ipot_t *pot, float ms[4], int *cycles, int *scorer_used);

/* Number of kernels this pot has launched since it was created. */
int ipot_launch_count(ipot_t *pot, long long *launches);

const char *ipot_strerror(int code);

/*
 * CaP scoring for callers that must not allocate device memory.  (The paper has
 * no counterpart: this is a packaging variant of the scoring step, computing the
 * same u_j as step 2 of ipot_score_and_compress() with the fp32 FMA kernels.)
 *
 * Who needs it: processes whose device memory is handed over, whole, to a
 * framework's own pool at start-up, where a later cudaMalloc can fail or eat
 * into that pool's reserve; and latency-sensitive loops, because cudaMalloc
 * and cudaFree synchronise the whole device and so stall every other stream.
 * No pot object is involved.  This call makes no cudaMalloc/cudaFree and calls
 * no allocating routine; its only scratch - one (max, 1/denominator) pair per
 * query row, handed from its first kernel launch to its second - is a fixed
 * array of IPOT_NOALLOC_MAX_ROWS pairs (512 KiB) that is part of the library
 * image, so every device that loads the library carries it until the process
 * exits.
 *
 *   Q       device [units][rows][d]          query rows of each unit (rows = G * cap_rows)
 *   K       device [units][k_unit_rows][d]   keys; the first N rows of each unit are scored
 *   scores  device [units][N] f32            output, fully overwritten
 *   dtype   IPOT_BF16 or IPOT_F32 (element type of Q and K); d as for ipot_create()
 *   cuda_stream  cudaStream_t (NULL = default stream); the call only queues work
 *
 * Limits and errors: units * rows > IPOT_NOALLOC_MAX_ROWS -> IPOT_E_LIMIT,
 * nothing is launched.  INVALID for NULL/misaligned pointers or bad sizes, CUDA
 * for runtime failures.
 * First use on a device: the first call made while a given device is current
 * looks up the array's device address (cudaGetSymbolAddress) and keeps it; make
 * that first call outside any stream capture.
 * Sharing: all calls on a device use the same array, and it keeps whatever the
 * last call left there.  Nothing has to be cleared, because each call writes
 * every entry it later reads; but two calls whose kernels can overlap on the
 * GPU (different streams, no ordering between them) race on it - order them.
 */
#define IPOT_NOALLOC_MAX_ROWS 65536
int ipot_cap_scores_noalloc(const void *Q, const void *K, float *scores, int units, int rows, int N, int d,
                            int k_unit_rows, int dtype, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* IPOT_H */
