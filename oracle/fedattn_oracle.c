/*
 * fedattn_oracle.c -- TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT PATH.
 *
 * A plain, slow, fp64 CPU statement of what the FedAttn attention step computes,
 * written from the paper's definitions.  Only the tests, the smoke check and the
 * benchmark's cpu_baseline / reference legs may call it.  It shares no code with
 * the CUDA library.
 *
 * Every attention result below is the direct definition: for one query row,
 * materialise the scaled logits over the allowed key set, subtract their maximum,
 * exponentiate, normalise, and take the weighted sum of the value rows.  No
 * blocking, no online softmax, no fusion.  OpenMP only spreads independent
 * (row, head) pairs over cores.
 *
 * Passages followed (paper sections / labelled equations):
 *   - scaled dot-product attention Softmax(Q K^T / sqrt(d)) V      : Sec. III-B, first equation
 *   - causal mask M                                                : Sec. III-B, mask equation.
 *       The printed case split (0 if i <= j) contradicts the text's "each token can
 *       only attend to preceding tokens"; the reading taken is: key j is allowed
 *       for query i iff j <= i (self included).
 *   - participant partition L_n, Pi_n, L = sum L_n                 : Sec. IV-A
 *   - local attention o_n = Attention(q_n, k_n, v_n)               : Sec. IV-B Phase I, eq. update_local_o
 *   - KV aggregation [K V] = sum_n Pi_n [k_n v_n] (concatenation)  : Sec. IV-B Phase II, eq. update_global_kv_H
 *   - global attention o_n = Attention(q_n, K, V)                  : Sec. IV-B Phase II, eq. update_local_o_H
 *       mask: causal on the global token index (so that sync at every block equals
 *       centralised attention, Remark after Corollary 1)
 *   - adaptive / sparse KV aggregation pi_n(t), L'_n(t) subset L_n : Sec. V, Observation "Aggregation method"
 *       dropped rows are removed (the text's "reduced dimensionality"), survivors keep
 *       their global position for the causal test
 *   - KV caches and decoding                                       : Sec. IV-C, Sec. III-C
 *
 * Layouts: Q [L, Hq, d]; K, V [L, Hkv, d] (token-major) or [Hkv, Lkv, d] (head-major,
 * sparse aggregation), always with d contiguous.  Query head h reads KV head
 * h / (Hq / Hkv).  All floating-point inputs and outputs are double.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int fedattn_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---- Sec. IV-A: off_n = sum_{n' < n} L_n', off_N = L ------------------------------ */
void fedattn_oracle_offsets(const int32_t *seqlens, int32_t n_participants, int32_t *off)
{
    off[0] = 0;
    for (int32_t n = 0; n < n_participants; ++n)
        off[n + 1] = off[n] + seqlens[n];
}

/*
 * One query row against an explicit list of allowed key rows.
 *   logits_j = scale * <q, K[allowed_j]>,  p = softmax(logits),  o = sum_j p_j V[allowed_j]
 *   lse = max + log(sum_j exp(logits_j - max))   (natural log of the scaled logits)
 * Empty allowed set: o = 0, lse = -inf.
 * krow(j) = K + j * kv_tok_stride ; same for V.
 */
static void attend_row(const double *q, const double *K, const double *V, int64_t kv_tok_stride,
                       const int64_t *allowed, int64_t n_allowed, int32_t d, double scale,
                       double *o, double *lse, double *logits /* scratch [n_allowed] */)
{
    for (int32_t c = 0; c < d; ++c)
        o[c] = 0.0;
    if (n_allowed == 0) {
        if (lse)
            *lse = -INFINITY;
        return;
    }
    double mx = -INFINITY;
    for (int64_t a = 0; a < n_allowed; ++a) {
        const double *kr = K + allowed[a] * kv_tok_stride;
        double s = 0.0;
        for (int32_t c = 0; c < d; ++c)
            s += q[c] * kr[c];
        logits[a] = s * scale;
        if (logits[a] > mx)
            mx = logits[a];
    }
    double denom = 0.0;
    for (int64_t a = 0; a < n_allowed; ++a) {
        logits[a] = exp(logits[a] - mx);
        denom += logits[a];
    }
    for (int64_t a = 0; a < n_allowed; ++a) {
        const double p = logits[a] / denom;
        const double *vr = V + allowed[a] * kv_tok_stride;
        for (int32_t c = 0; c < d; ++c)
            o[c] += p * vr[c];
    }
    if (lse)
        *lse = mx + log(denom);
}

/*
 * Local attention (Phase I, eq. update_local_o).  Row i of segment n (off_n <= i < off_{n+1})
 * may attend keys { j : off_n <= j <= i } when causal, or the whole segment otherwise.
 * rows: optional list of packed row indices to compute (NULL => all L rows, n_rows = L).
 * o: [n_rows, Hq, d]; lse: [n_rows, Hq] (nullable).
 */
void fedattn_oracle_local(const double *q, const double *k, const double *v,
                          const int32_t *off, int32_t n_participants,
                          int32_t hq, int32_t hkv, int32_t d, double scale, int32_t causal,
                          const int64_t *rows, int64_t n_rows, double *o, double *lse)
{
    const int32_t g = hq / hkv;
    const int64_t L = off[n_participants];
#pragma omp parallel
    {
        int64_t *allowed = (int64_t *)malloc(sizeof(int64_t) * (size_t)(L > 0 ? L : 1));
        double *logits = (double *)malloc(sizeof(double) * (size_t)(L > 0 ? L : 1));
#pragma omp for schedule(dynamic, 1) collapse(2)
        for (int64_t r = 0; r < n_rows; ++r) {
            for (int32_t h = 0; h < hq; ++h) {
                const int64_t i = rows ? rows[r] : r;
                int32_t n = 0;
                while (!(off[n] <= i && i < off[n + 1]))
                    ++n;
                int64_t na = 0;
                const int64_t last = causal ? i : (int64_t)off[n + 1] - 1;
                for (int64_t j = off[n]; j <= last; ++j)
                    allowed[na++] = j;
                const int32_t kvh = h / g;
                attend_row(q + (i * hq + h) * d, k + (int64_t)kvh * d, v + (int64_t)kvh * d,
                           (int64_t)hkv * d, allowed, na, d, scale,
                           o + (r * hq + h) * d, lse ? lse + r * hq + h : NULL, logits);
            }
        }
        free(allowed);
        free(logits);
    }
}

/*
 * Dense KV aggregation (eq. update_global_kv_H with contiguous index sets): participant n's
 * rows land at global rows off_n .. off_{n+1}-1.  kv_pos[j] = j; cu_kv = off.
 */
void fedattn_oracle_aggregate_concat(const double *const *k_parts, const double *const *v_parts,
                                     const int32_t *seqlens, int32_t n_participants,
                                     int32_t hkv, int32_t d,
                                     double *k_agg, double *v_agg, int32_t *kv_pos, int32_t *cu_kv)
{
    fedattn_oracle_offsets(seqlens, n_participants, cu_kv);
    const int64_t row = (int64_t)hkv * d;
    for (int32_t n = 0; n < n_participants; ++n) {
        for (int32_t j = 0; j < seqlens[n]; ++j) {
            const int64_t gj = (int64_t)cu_kv[n] + j;
            for (int64_t c = 0; c < row; ++c) {
                k_agg[gj * row + c] = k_parts[n][(int64_t)j * row + c];
                v_agg[gj * row + c] = v_parts[n][(int64_t)j * row + c];
            }
            kv_pos[gj] = (int32_t)gj;
        }
    }
}

/*
 * Key-norm top-k selection for one participant (the "critical KVs" of the sparse KV
 * exchange, with the squared L2 norm of the key row as the criticality score).
 *   score(j, head) = sum_{c=0}^{d-1} k[j, head, c]^2, accumulated in fp64 in increasing c
 *   order: larger score first; equal scores => lower token index first
 *   the k_sel winners are returned sorted ascending by token index.
 * k_part: [L_n, Hkv, d]; sel_idx: [Hkv, k_sel]; scores_out: nullable [Hkv, L_n].
 */
typedef struct {
    double score;
    int32_t idx;
} scored_t;

static int cmp_score_desc_idx_asc(const void *a, const void *b)
{
    const scored_t *x = (const scored_t *)a, *y = (const scored_t *)b;
    if (x->score > y->score) return -1;
    if (x->score < y->score) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);
}

static int cmp_i32(const void *a, const void *b)
{
    const int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

void fedattn_oracle_topk_knorm(const double *k_part, int32_t len, int32_t hkv, int32_t d,
                               int32_t k_sel, int32_t *sel_idx, double *scores_out)
{
    scored_t *sc = (scored_t *)malloc(sizeof(scored_t) * (size_t)(len > 0 ? len : 1));
    for (int32_t h = 0; h < hkv; ++h) {
        for (int32_t j = 0; j < len; ++j) {
            const double *kr = k_part + ((int64_t)j * hkv + h) * d;
            double s = 0.0;
            for (int32_t c = 0; c < d; ++c)
                s += kr[c] * kr[c];
            sc[j].score = s;
            sc[j].idx = j;
            if (scores_out)
                scores_out[(int64_t)h * len + j] = s;
        }
        qsort(sc, (size_t)len, sizeof(scored_t), cmp_score_desc_idx_asc);
        for (int32_t t = 0; t < k_sel; ++t)
            sel_idx[(int64_t)h * k_sel + t] = sc[t].idx;
        qsort(sel_idx + (int64_t)h * k_sel, (size_t)k_sel, sizeof(int32_t), cmp_i32);
    }
    free(sc);
}

/*
 * Sparse / adaptive KV aggregation (pi_n(t) with L'_n(t) given per KV head).
 * For KV head h the output row block of participant n is cu_kv[n] .. cu_kv[n+1]-1 and holds
 * the rows sel_idx[h, cu_kv[n] + t] (local indices, ascending) of k_n, v_n.
 *   k_agg, v_agg: [Hkv, total_sel, d]   (head-major; total_sel = sum_n k_sel[n])
 *   kv_pos:       [Hkv, total_sel]      global position off_n + local index
 *   cu_kv:        [N+1]                 prefix sum of k_sel  (k_sel[n] = 0 drops participant n)
 */
void fedattn_oracle_aggregate_indexed(const double *const *k_parts, const double *const *v_parts,
                                      const int32_t *seqlens, const int32_t *k_sel,
                                      int32_t n_participants, int32_t hkv, int32_t d,
                                      const int32_t *sel_idx /* [Hkv, total_sel] */,
                                      double *k_agg, double *v_agg, int32_t *kv_pos, int32_t *cu_kv)
{
    int32_t *off = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_participants + 1));
    fedattn_oracle_offsets(seqlens, n_participants, off);
    fedattn_oracle_offsets(k_sel, n_participants, cu_kv);
    const int64_t total = cu_kv[n_participants];
    for (int32_t h = 0; h < hkv; ++h) {
        for (int32_t n = 0; n < n_participants; ++n) {
            for (int32_t t = 0; t < k_sel[n]; ++t) {
                const int64_t out = (int64_t)h * total + cu_kv[n] + t;
                const int32_t j = sel_idx[out];
                for (int32_t c = 0; c < d; ++c) {
                    k_agg[out * d + c] = k_parts[n][((int64_t)j * hkv + h) * d + c];
                    v_agg[out * d + c] = v_parts[n][((int64_t)j * hkv + h) * d + c];
                }
                kv_pos[out] = off[n] + j;
            }
        }
    }
    free(off);
}

/*
 * Global (sync) attention (eq. update_local_o_H).  Query row i has global position
 * p_i = q_pos ? q_pos[i] : i.  Key row j of KV head kvh has position
 * kv_pos ? kv_pos[kvh * kv_pos_head_stride + j] : j, and is allowed iff position <= p_i
 * (or always, when causal == 0).
 * K element (j, kvh, c) sits at j * kv_tok_stride + kvh * kv_head_stride + c.
 * rows / o / lse as in fedattn_oracle_local.
 */
void fedattn_oracle_sync(const double *q, int64_t n_q, const int32_t *q_pos,
                         const double *k_agg, const double *v_agg, int64_t total_kv,
                         int64_t kv_tok_stride, int64_t kv_head_stride,
                         const int32_t *kv_pos, int64_t kv_pos_head_stride,
                         int32_t hq, int32_t hkv, int32_t d, double scale, int32_t causal,
                         const int64_t *rows, int64_t n_rows, double *o, double *lse)
{
    const int32_t g = hq / hkv;
    (void)n_q;
#pragma omp parallel
    {
        int64_t *allowed = (int64_t *)malloc(sizeof(int64_t) * (size_t)(total_kv > 0 ? total_kv : 1));
        double *logits = (double *)malloc(sizeof(double) * (size_t)(total_kv > 0 ? total_kv : 1));
#pragma omp for schedule(dynamic, 1) collapse(2)
        for (int64_t r = 0; r < n_rows; ++r) {
            for (int32_t h = 0; h < hq; ++h) {
                const int64_t i = rows ? rows[r] : r;
                const int64_t p_i = q_pos ? q_pos[i] : i;
                const int32_t kvh = h / g;
                int64_t na = 0;
                for (int64_t j = 0; j < total_kv; ++j) {
                    const int64_t p_j = kv_pos ? kv_pos[kvh * kv_pos_head_stride + j] : j;
                    if (!causal || p_j <= p_i)
                        allowed[na++] = j;
                }
                attend_row(q + (i * hq + h) * d, k_agg + kvh * kv_head_stride,
                           v_agg + kvh * kv_head_stride, kv_tok_stride, allowed, na, d, scale,
                           o + (r * hq + h) * d, lse ? lse + r * hq + h : NULL, logits);
            }
        }
        free(allowed);
        free(logits);
    }
}

/*
 * Sync block with sparse KV exchange as the paper's experiment describes it (Sec. VI, the
 * discussion of the sparsity-ratio figure: every participant keeps self-attention over its own
 * complete segment, only what it receives from the others is sparsified): row i of participant
 * n attends
 *     A = its own keys  { j : off_n <= j <= i }  (causal)  or the whole segment (causal == 0), and
 *     B = the exchanged keys of the OTHER participants,
 *         { t outside [cu_kv[n], cu_kv[n+1]) : kv_pos[kvh][t] <= i }  (causal on the global
 *         position), or every such t when causal == 0 (Sec. III-B: the attention operator stands
 *         for the masked or the bidirectional form),
 * with one softmax over A u B.  k, v: packed local tensors [L, Hkv, d]; k_agg, v_agg: head-major
 * aggregate [Hkv, T, d] with kv_pos [Hkv, T] and participant ranges cu_kv [N+1].
 * rows / o / lse as in fedattn_oracle_local.
 */
void fedattn_oracle_sync_exchange(const double *q, const double *k, const double *v,
                                  const int32_t *off, int32_t n_participants,
                                  const double *k_agg, const double *v_agg, const int32_t *kv_pos,
                                  const int32_t *cu_kv, int64_t total_kv,
                                  int32_t hq, int32_t hkv, int32_t d, double scale, int32_t causal,
                                  const int64_t *rows, int64_t n_rows, double *o, double *lse)
{
    const int32_t g = hq / hkv;
    const int64_t L = off[n_participants];
#pragma omp parallel
    {
        const size_t cap = (size_t)(L + total_kv > 0 ? L + total_kv : 1);
        double *logits = (double *)malloc(sizeof(double) * cap);
        const double **vrow = (const double **)malloc(sizeof(double *) * cap);
#pragma omp for schedule(dynamic, 1) collapse(2)
        for (int64_t r = 0; r < n_rows; ++r) {
            for (int32_t h = 0; h < hq; ++h) {
                const int64_t i = rows ? rows[r] : r;
                int32_t n = 0;
                while (!(off[n] <= i && i < off[n + 1]))
                    ++n;
                const int32_t kvh = h / g;
                const double *qr = q + (i * hq + h) * d;
                double *orow = o + (r * hq + h) * d;
                int64_t na = 0;
                double mx = -INFINITY;
                const int64_t last_own = causal ? i : (int64_t)off[n + 1] - 1;
                for (int64_t j = off[n]; j <= last_own; ++j) {     /* set A */
                    const double *kr = k + (j * hkv + kvh) * d;
                    double s = 0.0;
                    for (int32_t c = 0; c < d; ++c)
                        s += qr[c] * kr[c];
                    logits[na] = s * scale;
                    vrow[na] = v + (j * hkv + kvh) * d;
                    if (logits[na] > mx)
                        mx = logits[na];
                    ++na;
                }
                for (int64_t t = 0; t < total_kv; ++t) {           /* set B */
                    if (t >= cu_kv[n] && t < cu_kv[n + 1])
                        continue;
                    if (causal && kv_pos[(int64_t)kvh * total_kv + t] > i)
                        continue;
                    const double *kr = k_agg + ((int64_t)kvh * total_kv + t) * d;
                    double s = 0.0;
                    for (int32_t c = 0; c < d; ++c)
                        s += qr[c] * kr[c];
                    logits[na] = s * scale;
                    vrow[na] = v_agg + ((int64_t)kvh * total_kv + t) * d;
                    if (logits[na] > mx)
                        mx = logits[na];
                    ++na;
                }
                for (int32_t c = 0; c < d; ++c)
                    orow[c] = 0.0;
                double denom = 0.0;
                for (int64_t a = 0; a < na; ++a) {
                    logits[a] = exp(logits[a] - mx);
                    denom += logits[a];
                }
                for (int64_t a = 0; a < na; ++a) {
                    const double p = logits[a] / denom;
                    for (int32_t c = 0; c < d; ++c)
                        orow[c] += p * vrow[a][c];
                }
                if (lse)
                    lse[r * hq + h] = mx + log(denom);            /* A is never empty: the row itself */
            }
        }
        free(logits);
        free(vrow);
    }
}

/*
 * Decode step (Sec. IV-C): one new query token per participant, later than every cached
 * row, so the whole cache is allowed.
 *   sync == 0: participant n reads its own cache k_cache + n * cache_stride_participant,
 *              rows 0 .. kv_len[n]-1, layout [cap, Hkv, d]
 *   sync == 1: every participant reads the shared global cache, rows 0 .. kv_len[0]-1
 * q, o: [N, Hq, d]; lse: [N, Hq] (nullable).
 */
void fedattn_oracle_decode(const double *q, const double *k_cache, const double *v_cache,
                           int64_t cache_stride_participant, const int32_t *kv_len, int32_t sync,
                           int32_t n_participants, int32_t hq, int32_t hkv, int32_t d, double scale,
                           double *o, double *lse)
{
    const int32_t g = hq / hkv;
    int64_t max_len = 1;
    for (int32_t n = 0; n < (sync ? 1 : n_participants); ++n)
        if (kv_len[n] > max_len)
            max_len = kv_len[n];
#pragma omp parallel
    {
        int64_t *allowed = (int64_t *)malloc(sizeof(int64_t) * (size_t)max_len);
        double *logits = (double *)malloc(sizeof(double) * (size_t)max_len);
#pragma omp for schedule(dynamic, 1) collapse(2)
        for (int32_t n = 0; n < n_participants; ++n) {
            for (int32_t h = 0; h < hq; ++h) {
                const int64_t len = sync ? kv_len[0] : kv_len[n];
                const int64_t base = sync ? 0 : (int64_t)n * cache_stride_participant;
                for (int64_t j = 0; j < len; ++j)
                    allowed[j] = j;
                const int32_t kvh = h / g;
                attend_row(q + ((int64_t)n * hq + h) * d, k_cache + base + (int64_t)kvh * d,
                           v_cache + base + (int64_t)kvh * d, (int64_t)hkv * d, allowed, len, d,
                           scale, o + ((int64_t)n * hq + h) * d,
                           lse ? lse + (int64_t)n * hq + h : NULL, logits);
            }
        }
        free(allowed);
        free(logits);
    }
}
