/*
 * CPU checker for the CCD compression cycle of InfiniPot (arxiv 2410.01518).
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, double precision; one loop per
 * definition, no blocking, no fusion, no reordering.  It shares no code with
 * the CUDA library and must never be called from it; only the tests, the smoke
 * check and the CPU-baseline leg of the benchmark use it.
 *
 * What each function follows:
 *   ora_token_novelty  Sec. 3.3.2, Eq. 3 (the Appendix B listing computes it as a per-token
 *                    cross-entropy without reduction): n_t = -log softmax(logits_t)[x_t]
 *   ora_nuc_top      Sec. 3.3.3: the T slots with the highest NuC score are taken first
 *   ora_cap_scores   Sec. 3.3.1, Eq. 2: sum over the CaP query rows of the
 *                    self-attention probability towards every pot key
 *   ora_select       Sec. 3.3.3 + Appendix B "Combine NuC and CaP" / "Final
 *                    Token Selection": NuC slots first, the remaining |C|-T
 *                    slots by CaP score, per head
 *   ora_gather       Appendix B "KV-cache compression": K and V rows of the
 *                    retained slots
 *   ora_cap_scores_incl  the variant the Appendix B listing spells out: the CaP
 *                    queries attend to the pot keys AND, causally, to the CaP's
 *                    own keys; the CaP columns are then cut away, so they only
 *                    take probability mass from the pot columns
 *   ora_rope_rows    Sec. 3.4 (CR-RoPE): keys are kept without rotary embedding and get it
 *                    at their position inside the pot, 0 .. len-1
 *   ora_decode_attention  generation over the pot (Sec. 3.3.1 notes that the heads keep different
 *                    tokens; Sec. 4.5 measures generation at a fixed pot): plain softmax attention
 *                    of one new query per head over the unit's own rows
 *   ora_cycle        the four steps over every (layer, stream, kv-head) unit
 *   ora_cycle_cap    the same with the CaP-inclusive scores
 *
 * Readings where the paper is silent (each listed in the design notes):
 *   - every CaP row normalises over the N pot keys only (CaP keys are not in
 *     the pot), so each softmax row sums to 1 over the context slots;
 *   - logits are scaled by 1/sqrt(d);
 *   - with grouped-query attention the G query heads that share a KV head are
 *     summed like additional CaP rows (Eq. 2 is a plain sum);
 *   - the CaP top-(|C|-T) is taken among slots not already taken by NuC, so
 *     exactly |C| slots survive;
 *   - ties: the lower slot index wins, in both rankings;
 *   - survivors keep their original order (ascending slot index);
 *   - CR-RoPE: the paper gives no rotary details.  The caller supplies cos/sin per (position,
 *     frequency) in the storage type; channel pairs are (c, c + d/2) ("half") or (2c, 2c + 1)
 *     ("interleaved"); the pair is multiplied as a complex number by cos + i sin in double
 *     precision and rounded once to the storage type (nearest even).  A CUDA path that evaluates
 *     the same product in single precision agrees with it bit for bit except where the exact
 *     value lies within its rounding error of a rounding boundary; the tests bound that.
 *
 *   - CaP-inclusive variant: CaP row i (0-based, within its query head) sees the
 *     CaP keys 0..i of its KV head (causal mask), all of them after every pot key;
 * Parity pins (tests/test_oracle_pins.py): row sums = 1, column-sum total =
 * G*P, closed forms (Q = 0, equal keys, N = 1, one dominant key), slot
 * permutation equivariance, P=G=1 against an independent library softmax,
 * brute-force subset enumeration for the selection on tiny pots, NuC-only and
 * CaP-only special cases, byte-wise gather identities.  CaP-inclusive variant:
 * Q = 0 closed form G * sum_i 1/(N+i+1), masked library softmax over the N+P
 * columns, far-away CaP keys reduce it to ora_cap_scores, a later CaP key never
 * changes an earlier row.  Token novelty: uniform logits give log V, V = 2 is a
 * softplus, a constant added to a row changes nothing, library cross-entropy.
 * Rotary rows: position 0 is the identity, exact small cases, exact rational arithmetic with
 * a brute-force search for the nearest storage value, library complex multiplication, pair
 * norms, the score of a rotated query and key depends on the position difference only, the
 * two pairings are one channel permutation apart.
 * Decode attention: one key returns its value, equal keys the mean value, library attention
 * and log-sum-exp, slot permutation invariance.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ---- ranking helper: indices sorted by (value descending, index ascending) ---- */
typedef struct { double v; int j; } ora_pair;

static int ora_cmp_desc(const void *a, const void *b)
{
    const ora_pair *x = (const ora_pair *)a, *y = (const ora_pair *)b;
    if (x->v > y->v) return -1;
    if (x->v < y->v) return 1;
    return (x->j > y->j) - (x->j < y->j);
}

static int ora_cmp_int(const void *a, const void *b)
{
    int x = *(const int *)a, y = *(const int *)b;
    return (x > y) - (x < y);
}

/*
 * Eq. 3: novelty of token t = -log P(x_t | prefix) = log sum_v exp(z_tv) - z_t,label for the
 * model's logits z ([n][V], row stride V).  A label outside [0, V) gives 0 (such a token is
 * ignored, as a padding position would be).
 */
void ora_token_novelty(const double *logits, const int *labels, long n, int V, double *out)
{
    for (long t = 0; t < n; ++t) {
        const double *z = logits + (size_t)t * V;
        if (labels[t] < 0 || labels[t] >= V) { out[t] = 0.0; continue; }
        double m = -INFINITY;
        for (int v = 0; v < V; ++v) if (z[v] > m) m = z[v];
        double Z = 0.0;
        for (int v = 0; v < V; ++v) Z += exp(z[v] - m);
        out[t] = (m + log(Z)) - z[labels[t]];
    }
}

/* The T slots with the largest aux value (ties: lower slot first), returned ascending. */
void ora_nuc_top(const double *aux, int N, int T, int *out)
{
    ora_pair *p = (ora_pair *)malloc(sizeof(ora_pair) * (size_t)(N > 0 ? N : 1));
    for (int j = 0; j < N; ++j) { p[j].v = aux[j]; p[j].j = j; }
    qsort(p, (size_t)N, sizeof(ora_pair), ora_cmp_desc);
    for (int r = 0; r < T; ++r) out[r] = p[r].j;
    qsort(out, (size_t)T, sizeof(int), ora_cmp_int);
    free(p);
}

/*
 * Eq. 2 for one KV head.  Q holds the M = G*P query rows that attend to this
 * head's keys ([M][d]); K holds the N pot keys ([N][d]).  For every row:
 * s_j = q.k_j / sqrt(d), p_j = exp(s_j - max) / sum, and u_j += p_j.
 * If row_sums is not NULL it receives sum_j p_j of every row (should be 1).
 */
void ora_cap_scores(const double *Q, const double *K, int M, int N, int d,
                    double *u, double *row_sums)
{
    double *s = (double *)malloc(sizeof(double) * (size_t)(N > 0 ? N : 1));
    const double scale = 1.0 / sqrt((double)d);
    for (int j = 0; j < N; ++j) u[j] = 0.0;
    for (int i = 0; i < M; ++i) {
        const double *q = Q + (size_t)i * d;
        double m = -INFINITY;
        for (int j = 0; j < N; ++j) {
            const double *k = K + (size_t)j * d;
            double acc = 0.0;
            for (int c = 0; c < d; ++c) acc += q[c] * k[c];
            s[j] = acc * scale;
            if (s[j] > m) m = s[j];
        }
        double Z = 0.0;
        for (int j = 0; j < N; ++j) { s[j] = exp(s[j] - m); Z += s[j]; }
        double rs = 0.0;
        for (int j = 0; j < N; ++j) { double p = s[j] / Z; u[j] += p; rs += p; }
        if (row_sums) row_sums[i] = rs;
    }
    free(s);
}

/*
 * Appendix B "Calculate Attention Score", read literally.  Row r of Q belongs to CaP
 * position i = r % P of one of the G query heads; Kc holds the P CaP keys of the KV
 * head ([P][d]).  The row's softmax runs over the N pot keys and the CaP keys 0..i;
 * only the pot columns are added into u.  pot_mass (may be NULL) receives, per row,
 * the probability that stayed on the pot columns (1 minus what the CaP keys took).
 */
void ora_cap_scores_incl(const double *Q, const double *K, const double *Kc, int M, int N, int d,
                         int P, double *u, double *pot_mass)
{
    double *s = (double *)malloc(sizeof(double) * (size_t)(N + P));
    const double scale = 1.0 / sqrt((double)d);
    for (int j = 0; j < N; ++j) u[j] = 0.0;
    for (int r = 0; r < M; ++r) {
        const double *q = Q + (size_t)r * d;
        const int i = r % P;          /* CaP position of this row */
        const int n = N + i + 1;      /* columns this row may see */
        double m = -INFINITY;
        for (int j = 0; j < n; ++j) {
            const double *k = (j < N) ? K + (size_t)j * d : Kc + (size_t)(j - N) * d;
            double acc = 0.0;
            for (int c = 0; c < d; ++c) acc += q[c] * k[c];
            s[j] = acc * scale;
            if (s[j] > m) m = s[j];
        }
        double Z = 0.0;
        for (int j = 0; j < n; ++j) { s[j] = exp(s[j] - m); Z += s[j]; }
        double pm = 0.0;
        for (int j = 0; j < N; ++j) { double p = s[j] / Z; u[j] += p; pm += p; }
        if (pot_mass) pot_mass[r] = pm;
    }
    free(s);
}

/* ---- storage <-> double.  bf16 = the upper half of a float; every bf16 and float value is a double ---- */
static double ora_load(const void *p, size_t i, int is_f32)
{
    if (is_f32) return (double)((const float *)p)[i];
    uint32_t w = (uint32_t)((const uint16_t *)p)[i] << 16;
    float f;
    memcpy(&f, &w, 4);
    return (double)f;
}

/* One rounding, to nearest (ties to even), from double to bf16: 8 significant bits, or a multiple of
 * 2^-133 below the normal range. */
static uint16_t ora_double_to_bf16(double v)
{
    float f;
    if (v == 0.0 || !isfinite(v)) {
        f = (float)v;
    } else {
        int e;
        (void)frexp(fabs(v), &e);                 /* |v| = m 2^e with m in [0.5, 1) */
        int qe = e - 8;
        if (qe < -133) qe = -133;
        const double q = ldexp(1.0, qe);
        f = (float)copysign(rint(fabs(v) / q) * q, v);   /* rint: nearest even; the result fits a float exactly */
    }
    uint32_t w;
    memcpy(&w, &f, 4);
    return (uint16_t)(w >> 16);
}

static void ora_store(void *p, size_t i, int is_f32, double v)
{
    if (is_f32) ((float *)p)[i] = (float)v;       /* one rounding to nearest even */
    else ((uint16_t *)p)[i] = ora_double_to_bf16(v);
}

/*
 * Sec. 3.4: rotary embedding of n rows of d channels; row r gets position pos[r].  cos_t and
 * sin_t are [positions][d/2] tables in the storage type.  interleaved = 0 pairs channel c with
 * c + d/2, 1 pairs 2c with 2c + 1; frequency index c in both.  Each pair (lo, hi) is the complex
 * number lo + i hi multiplied by cos + i sin, in double precision (the products of two storage
 * values are exact there), rounded once to the storage type.  in and out may not overlap.
 * exact and mag (each may be NULL, [n][d] doubles) receive the unrounded result and
 * |lo cos| + |hi sin| resp. |hi cos| + |lo sin|: the size of the terms whose difference the
 * result is, which bounds what an evaluation in a narrower type can lose to cancellation.
 */
void ora_rope_rows(const void *in, void *out, const int *pos, int n, int d, int is_f32,
                   const void *cos_t, const void *sin_t, int interleaved, double *exact, double *mag)
{
    const int half = d / 2;
    for (int r = 0; r < n; ++r) {
        for (int c = 0; c < half; ++c) {
            const size_t ilo = (size_t)r * d + (interleaved ? 2 * c : c);
            const size_t ihi = (size_t)r * d + (interleaved ? 2 * c + 1 : c + half);
            const double lo = ora_load(in, ilo, is_f32), hi = ora_load(in, ihi, is_f32);
            const double cs = ora_load(cos_t, (size_t)pos[r] * half + c, is_f32);
            const double sn = ora_load(sin_t, (size_t)pos[r] * half + c, is_f32);
            const double re = lo * cs - hi * sn, im = hi * cs + lo * sn;
            ora_store(out, ilo, is_f32, re);
            ora_store(out, ihi, is_f32, im);
            if (exact) { exact[ilo] = re; exact[ihi] = im; }
            if (mag) { mag[ilo] = fabs(lo * cs) + fabs(hi * sn); mag[ihi] = fabs(hi * cs) + fabs(lo * sn); }
        }
    }
}

/*
 * Attention of G new queries (the query heads of one KV head, [G][d]) over the N rows of a unit:
 * out[h] = sum_j softmax_j(q_h . k_j / sqrt(d)) v_j, lse[h] = log sum_j exp(q_h . k_j / sqrt(d))
 * (lse lets a caller merge this with attention over tokens that are not in the pot).
 */
void ora_decode_attention(const double *Q, const double *K, const double *V, int G, int N, int d,
                          double *out, double *lse)
{
    double *s = (double *)malloc(sizeof(double) * (size_t)(N > 0 ? N : 1));
    const double scale = 1.0 / sqrt((double)d);
    for (int h = 0; h < G; ++h) {
        const double *q = Q + (size_t)h * d;
        double m = -INFINITY;
        for (int j = 0; j < N; ++j) {
            double acc = 0.0;
            for (int c = 0; c < d; ++c) acc += q[c] * K[(size_t)j * d + c];
            s[j] = acc * scale;
            if (s[j] > m) m = s[j];
        }
        double Z = 0.0;
        for (int j = 0; j < N; ++j) { s[j] = exp(s[j] - m); Z += s[j]; }
        for (int c = 0; c < d; ++c) {
            double o = 0.0;
            for (int j = 0; j < N; ++j) o += (s[j] / Z) * V[(size_t)j * d + c];
            out[(size_t)h * d + c] = o;
        }
        if (lse) lse[h] = m + log(Z);
    }
    free(s);
}

/*
 * Per-head selection.  nuc[0..T) are the NuC slots of the stream (they are kept
 * in every head); of the other slots the R = keep - T with the largest u are
 * kept (ties: lower slot first).  idx[0..keep) is returned ascending.
 */
void ora_select(const double *u, int N, const int *nuc, int T, int keep, int *idx)
{
    char *taken = (char *)calloc((size_t)(N > 0 ? N : 1), 1);
    ora_pair *p = (ora_pair *)malloc(sizeof(ora_pair) * (size_t)(N > 0 ? N : 1));
    int n = 0, c = 0;
    for (int r = 0; r < T; ++r) { taken[nuc[r]] = 1; idx[c++] = nuc[r]; }
    for (int j = 0; j < N; ++j) if (!taken[j]) { p[n].v = u[j]; p[n].j = j; ++n; }
    qsort(p, (size_t)n, sizeof(ora_pair), ora_cmp_desc);
    for (int r = 0; r < keep - T; ++r) idx[c++] = p[r].j;
    qsort(idx, (size_t)keep, sizeof(int), ora_cmp_int);
    free(p);
    free(taken);
}

/* out[r] = rows[idx[r]], byte-wise. */
void ora_gather(const uint8_t *rows, size_t row_bytes, const int *idx, int keep, uint8_t *out)
{
    for (int r = 0; r < keep; ++r)
        memcpy(out + (size_t)r * row_bytes, rows + (size_t)idx[r] * row_bytes, row_bytes);
}

/*
 * One whole cycle over n_units independent (layer, stream, kv-head) units.
 *   Qd   [n_units][M][d] double   the M = G*P query rows of the unit's KV head
 *                                 (the G query heads h with h / G == kv-head,
 *                                 P CaP rows each)
 *   Kd   [n_units][N][d] double   the unit's pot keys
 *   Kb,Vb[n_units][N][row_bytes]  raw storage bytes of the unit's pot rows
 *   aux  [B][N] double            per-slot novelty, shared by all heads and
 *                                 layers of a stream
 *   stream_of[n_units]            which stream (row of aux) each unit belongs to
 * Outputs:
 *   u_out [n_units][N], idx_out [n_units][keep],
 *   Kout, Vout [n_units][keep][row_bytes]  (may be NULL)
 * Units are independent; with OpenMP one thread takes one unit at a time.
 */
/* Kcd: [n_units][P][d] double CaP keys, or NULL for the context-only softmax of ora_cycle. */
void ora_cycle_cap(const double *Qd, const double *Kd, const double *Kcd, const uint8_t *Kb,
                   const uint8_t *Vb, const double *aux, const int *stream_of, int n_units, int B,
                   int M, int P, int d, int N, int keep, int T, size_t row_bytes,
                   double *u_out, int *idx_out, uint8_t *Kout, uint8_t *Vout)
{
    int *nuc = (int *)malloc(sizeof(int) * (size_t)B * (size_t)(T > 0 ? T : 1));
    for (int b = 0; b < B; ++b) ora_nuc_top(aux + (size_t)b * N, N, T, nuc + (size_t)b * T);
#pragma omp parallel for schedule(dynamic, 1)
    for (int t = 0; t < n_units; ++t) {
        const double *Q = Qd + (size_t)t * M * d;
        const double *K = Kd + (size_t)t * N * d;
        double *u = u_out + (size_t)t * N;
        int *idx = idx_out + (size_t)t * keep;
        if (Kcd) ora_cap_scores_incl(Q, K, Kcd + (size_t)t * P * d, M, N, d, P, u, NULL);
        else ora_cap_scores(Q, K, M, N, d, u, NULL);
        ora_select(u, N, nuc + (size_t)stream_of[t] * T, T, keep, idx);
        if (Kout) ora_gather(Kb + (size_t)t * N * row_bytes, row_bytes, idx, keep,
                             Kout + (size_t)t * keep * row_bytes);
        if (Vout) ora_gather(Vb + (size_t)t * N * row_bytes, row_bytes, idx, keep,
                             Vout + (size_t)t * keep * row_bytes);
    }
    free(nuc);
}

void ora_cycle(const double *Qd, const double *Kd, const uint8_t *Kb, const uint8_t *Vb,
               const double *aux, const int *stream_of, int n_units, int B, int M, int d,
               int N, int keep, int T, size_t row_bytes,
               double *u_out, int *idx_out, uint8_t *Kout, uint8_t *Vout)
{
    ora_cycle_cap(Qd, Kd, NULL, Kb, Vb, aux, stream_of, n_units, B, M, 1, d, N, keep, T, row_bytes,
                  u_out, idx_out, Kout, Vout);
}

/* Thread count used by ora_cycle (1 when built without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
void ora_set_threads(int n) { if (n > 0) omp_set_num_threads(n); }
int ora_max_threads(void) { return omp_get_max_threads(); }
#else
void ora_set_threads(int n) { (void)n; }
int ora_max_threads(void) { return 1; }
#endif
