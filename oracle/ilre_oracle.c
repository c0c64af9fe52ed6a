/*
 * CPU oracle for the ILRe token-recall path.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, double-precision restatement of what the paper defines:
 *   - Eq. 4: attention of the query part over the cached context keys of the retrieval
 *     layer, softmax over the context axis, scale 1/sqrt(d_h), no mask;
 *   - Eq. 5: element-wise maximum over heads and query tokens -> one score per position;
 *   - Algorithm 1 ("Context Allocation"): strided max pooling, stride-1 window pooling,
 *     top-K_m per (max, window) combination, per-combination quota with de-duplication,
 *     ascending sort.
 * Only the tests, the smoke check and the bench's CPU-baseline leg may call this file; it
 * shares no code with the CUDA library and the CUDA library never calls it.
 *
 * Readings where the paper is silent (each is also listed in the design notes):
 *   R1  reduction over (head, query token) is a max over all query heads and tokens (Eq. 5).
 *   R2  softmax runs over the L context keys only, sink keys included, no mask (Eq. 4).
 *   R3  GQA: query head h reads kv head h / (n_q_heads / n_kv_heads).
 *   R4  "without sink part": softmax over all keys first, then positions < n_sink are
 *       dropped from pooling and returned unconditionally; they use no budget.
 *   R5  strided max pooling is ceil-mode: a shorter last cell.
 *   R6  window pooling keeps the length; zero padding; the average always divides by n.
 *   R7  window of size n at cell c covers [c - n/2, c - n/2 + n - 1] (integer division).
 *   R8  K_m = floor(B/m) + 1, plus one more when a partial tail cell exists, clipped to the
 *       number of cells.
 *   R9  B_c = floor(B/N_c); the first (B mod N_c) combinations in loop order get one more.
 *   R10 combination order: max sizes outer, window sizes inner, each in the order given.
 *   R11 ranking is (value descending, cell index ascending); inside a cell tokens are taken
 *       in ascending position; a quota may end inside a cell.
 *   R12 a selected cell c stands for the m tokens of max-pool cell c only.
 *
 * Pins (tests/test_oracle_*.py): softmax rows sum to one; identical keys give 1/L; a
 * single head and query token reduces to a library softmax; closed-form two-key case for
 * the 1/sqrt(d) scale; GQA mapping against a library einsum; brute-force pooling and
 * ranking on tiny arrays; size-1 pooling is the identity; monotone arrays; the SnapKV
 * special case (one size-1 max kernel, one average kernel) equals a plain top-B; a
 * hand-worked Algorithm 1 example; quota/unique/ascending invariants; needle recovery.
 * The paper prints no worked numerical example of this path, so none is pinned.
 *
 * Also here: Eq. 7, the re-rotation of the retrieval layer's cached keys under Dual Chunk
 * Attention (ilre_oracle_dca_rerope), with these readings:
 *   R13 chunks: chunk 1 holds the n_sink sink tokens plus `chunk` tokens, every later chunk
 *       `chunk` tokens (the last one possibly fewer); N_C = ceil((L - n_sink) / chunk).
 *   R14 D_i = (N_C - 1 - i) * chunk positions for i < N_C - 1, nothing for the last two chunks.
 *   R15 R(D) is the RoPE rotation by D positions in the rotate-half layout: channel pair
 *       (c, c + d/2) turns by the angle D * theta^(-2c/d).
 * Pins (tests/test_oracle_dca.py): a hand-computed pair rotation; pair norms are kept; the
 * last two chunks are untouched; rotating a key that carries RoPE at position p gives the
 * key with RoPE at position p + D (against an independent RoPE routine); the logit identity
 * q . R(D) k = (R(-D) q) . k; keys that differ only by whole chunks become equal.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_double(uint16_t v)
{
    uint32_t bits = ((uint32_t)v) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/* logit of query row (i, h) against key t of kv head g: Eq. 4 numerator, scaled. */
static double logit(const double *q, const double *k, int d)
{
    double acc = 0.0;
    for (int c = 0; c < d; ++c) acc += q[c] * k[c];
    return acc / sqrt((double)d);
}

/*
 * Row statistics of Eq. 4's softmax for a list of rows.
 *   K  bf16 [L][n_kv][d], Q bf16 [q_len][n_q][d];
 *   rows[j] = i * n_q + h names query token i, head h;
 *   row_max[j] = max_t s, row_sum[j] = sum_t exp(s - row_max).
 * Returns 0, or -1 on allocation failure.
 */
int ilre_oracle_row_stats(const uint16_t *K, int64_t L, int n_kv,
                          const uint16_t *Q, int q_len, int n_q, int d,
                          const int32_t *rows, int n_rows,
                          double *row_max, double *row_sum)
{
    (void)q_len;
    const int group = n_q / n_kv;
    int failed = 0;
    for (int g = 0; g < n_kv; ++g) {
        int any = 0;
        for (int j = 0; j < n_rows; ++j)
            if ((rows[j] % n_q) / group == g) any = 1;
        if (!any) continue;
        double *Kg = (double *)malloc((size_t)L * d * sizeof(double));
        if (!Kg) return -1;
        for (int64_t t = 0; t < L; ++t)
            for (int c = 0; c < d; ++c)
                Kg[t * d + c] = bf16_to_double(K[(t * n_kv + g) * d + c]);
#pragma omp parallel for schedule(dynamic, 1)
        for (int j = 0; j < n_rows; ++j) {
            const int h = rows[j] % n_q;
            if (h / group != g) continue;
            double *s = (double *)malloc((size_t)L * sizeof(double));
            double q[1024];
            if (!s || d > 1024) { failed = 1; free(s); continue; }
            for (int c = 0; c < d; ++c) q[c] = bf16_to_double(Q[(int64_t)rows[j] * d + c]);
            double m = -INFINITY;
            for (int64_t t = 0; t < L; ++t) {
                s[t] = logit(q, Kg + t * d, d);
                if (s[t] > m) m = s[t];
            }
            double z = 0.0;
            for (int64_t t = 0; t < L; ++t) z += exp(s[t] - m);
            row_max[j] = m;
            row_sum[j] = z;
            free(s);
        }
        free(Kg);
    }
    return failed ? -1 : 0;
}

/*
 * Eq. 5 at a list of context positions, given the row statistics of ALL rows
 * (row index i * n_q + h):  A[t] = max_{h,i} exp(s - row_max) / row_sum.
 */
int ilre_oracle_scores_at(const uint16_t *K, int64_t L, int n_kv,
                          const uint16_t *Q, int q_len, int n_q, int d,
                          const double *row_max, const double *row_sum,
                          const int64_t *pos, int64_t n_pos, double *A)
{
    (void)L;
    const int group = n_q / n_kv;
    const int R = q_len * n_q;
    if (d > 1024) return -1;
    double *Qd = (double *)malloc((size_t)R * d * sizeof(double));
    if (!Qd) return -1;
    for (int64_t e = 0; e < (int64_t)R * d; ++e) Qd[e] = bf16_to_double(Q[e]);
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < n_pos; ++j) {
        const int64_t t = pos[j];
        double a = 0.0;
        for (int g = 0; g < n_kv; ++g) {
            double k[1024];
            for (int c = 0; c < d; ++c) k[c] = bf16_to_double(K[(t * n_kv + g) * d + c]);
            for (int i = 0; i < q_len; ++i)
                for (int hh = 0; hh < group; ++hh) {
                    const int r = i * n_q + g * group + hh;
                    const double s = logit(Qd + (int64_t)r * d, k, d);
                    const double p = exp(s - row_max[r]) / row_sum[r];
                    if (p > a) a = p;
                }
        }
        A[j] = a;
    }
    free(Qd);
    return 0;
}

/* Eq. 4 + Eq. 5 over the whole cache: A[L]; optional row_max / row_sum [q_len * n_q]. */
int ilre_oracle_scores(const uint16_t *K, int64_t L, int n_kv,
                       const uint16_t *Q, int q_len, int n_q, int d,
                       double *A, double *row_max_out, double *row_sum_out)
{
    const int R = q_len * n_q;
    int rc = -1;
    int32_t *rows = (int32_t *)malloc((size_t)R * sizeof(int32_t));
    int64_t *pos = (int64_t *)malloc((size_t)L * sizeof(int64_t));
    double *m = (double *)malloc((size_t)R * sizeof(double));
    double *z = (double *)malloc((size_t)R * sizeof(double));
    if (rows && pos && m && z) {
        for (int r = 0; r < R; ++r) rows[r] = r;
        for (int64_t t = 0; t < L; ++t) pos[t] = t;
        rc = ilre_oracle_row_stats(K, L, n_kv, Q, q_len, n_q, d, rows, R, m, z);
        if (rc == 0) rc = ilre_oracle_scores_at(K, L, n_kv, Q, q_len, n_q, d, m, z, pos, L, A);
        if (rc == 0 && row_max_out) memcpy(row_max_out, m, (size_t)R * sizeof(double));
        if (rc == 0 && row_sum_out) memcpy(row_sum_out, z, (size_t)R * sizeof(double));
    }
    free(rows); free(pos); free(m); free(z);
    return rc;
}

/* Algorithm 1, MaxPooling with size = stride = m over a[0..n): ceil mode (R5). */
int64_t ilre_oracle_maxpool(const double *a, int64_t n, int m, double *out)
{
    const int64_t len = (n + m - 1) / m;
    for (int64_t c = 0; c < len; ++c) {
        double v = -INFINITY;
        for (int64_t t = c * m; t < c * m + m && t < n; ++t)
            if (a[t] > v) v = a[t];
        out[c] = v;
    }
    return len;
}

/* Precision of the averaging window (the only rounded step of Algorithm 1): 0 = double (the
 * definition), 1 = single.  Which cells Algorithm 1 ranks first is an integer decision taken
 * from these sums; to compare such a decision with an implementation that averages in
 * single precision, both sides must round alike, so the oracle can also add the window left to
 * right in float and divide in float (inputs that are exact floats stay exact). */
static int g_avg_single = 0;
void ilre_oracle_avg_precision(int single) { g_avg_single = single ? 1 : 0; }

/* Algorithm 1, stride-1 window pooling of size n over p[0..len): op 0 = average, 1 = max
 * (R6, R7). */
void ilre_oracle_winpool(const double *p, int64_t len, int n, int op, double *out)
{
    for (int64_t c = 0; c < len; ++c) {
        const int64_t lo = c - n / 2;
        if (op == 0 && g_avg_single) {
            float acc = 0.0f;
            for (int64_t u = lo; u < lo + n; ++u)
                if (u >= 0 && u < len) acc += (float)p[u];
            out[c] = (double)(acc / (float)n);
        } else if (op == 0) {
            double acc = 0.0;
            for (int64_t u = lo; u < lo + n; ++u)
                if (u >= 0 && u < len) acc += p[u];
            out[c] = acc / (double)n;
        } else {
            double v = -INFINITY;
            for (int64_t u = lo; u < lo + n; ++u)
                if (u >= 0 && u < len && p[u] > v) v = p[u];
            out[c] = v;
        }
    }
}

typedef struct { double v; int64_t c; } ranked_t;

static int by_value_desc_then_cell(const void *x, const void *y)
{
    const ranked_t *a = (const ranked_t *)x, *b = (const ranked_t *)y;
    if (a->v > b->v) return -1;
    if (a->v < b->v) return 1;
    return (a->c > b->c) - (a->c < b->c);
}

/*
 * Algorithm 1 on a score array A[L] (positions 0..L-1 of the context).
 *   n_sink leading positions are put into I first and take no budget (R4);
 *   out_idx receives n_sink + budget ascending positions;
 *   optional per-combination diagnostics (arrays of n_max * n_win entries, may be NULL):
 *     quota[c], taken[c], last_value[c] = pooled value of the last cell that contributed a
 *     token, kth_value[c] = pooled value of the K_m-th ranked cell;
 *   optional comb_out[L] (may be NULL): for every position the index of the combination that
 *     allocated it, -1 for positions that were not allocated (sink positions included).
 * Returns 0; -1 allocation failure; -2 budget > L - n_sink or bad sizes; -3 if some
 * combination ran out of candidates before meeting its quota.
 */
int ilre_oracle_allocate(const double *A, int64_t L, int n_sink, int budget,
                         const int32_t *max_sizes, int n_max,
                         const int32_t *win_sizes, int n_win, int win_op,
                         int32_t *out_idx,
                         int32_t *quota_out, int32_t *taken_out,
                         double *last_value_out, double *kth_value_out, int32_t *comb_out)
{
    if (n_sink < 0 || budget < 0 || n_max < 1 || n_win < 1) return -2;
    const int64_t Lp = L - n_sink;                 /* length without the sink part */
    if (Lp < 0 || budget > Lp) return -2;
    for (int i = 0; i < n_max; ++i) if (max_sizes[i] < 1) return -2;
    for (int j = 0; j < n_win; ++j) if (win_sizes[j] < 1) return -2;

    unsigned char *in_I = (unsigned char *)calloc((size_t)(L > 0 ? L : 1), 1);
    double *P = (double *)malloc((size_t)(Lp > 0 ? Lp : 1) * sizeof(double));
    double *W = (double *)malloc((size_t)(Lp > 0 ? Lp : 1) * sizeof(double));
    ranked_t *rk = (ranked_t *)malloc((size_t)(Lp > 0 ? Lp : 1) * sizeof(ranked_t));
    if (!in_I || !P || !W || !rk) { free(in_I); free(P); free(W); free(rk); return -1; }

    int rc = 0;
    if (comb_out) for (int64_t t = 0; t < L; ++t) comb_out[t] = -1;
    for (int t = 0; t < n_sink; ++t) in_I[t] = 1;  /* I <- indices of the sink part */
    const double *Ap = A + n_sink;                 /* A^C without the sink part     */
    const int n_comb = n_max * n_win;
    int comb = 0;
    for (int i = 0; i < n_max; ++i) {
        const int m = max_sizes[i];
        const int64_t len = ilre_oracle_maxpool(Ap, Lp, m, P);
        int64_t K_m = budget / m + 1 + ((Lp % m) != 0 ? 1 : 0);          /* R8 */
        if (K_m > len) K_m = len;
        for (int j = 0; j < n_win; ++j, ++comb) {
            const int quota = budget / n_comb + (comb < budget % n_comb ? 1 : 0); /* R9 */
            ilre_oracle_winpool(P, len, win_sizes[j], win_op, W);
            for (int64_t c = 0; c < len; ++c) { rk[c].v = W[c]; rk[c].c = c; }
            qsort(rk, (size_t)len, sizeof(ranked_t), by_value_desc_then_cell);
            int taken = 0;
            double last_v = NAN;
            for (int64_t r = 0; r < K_m && taken < quota; ++r) {
                const int64_t c = rk[r].c;
                for (int64_t t = c * m; t < c * m + m && t < Lp && taken < quota; ++t) {
                    const int64_t posn = n_sink + t;
                    if (!in_I[posn]) {
                        in_I[posn] = 1; ++taken; last_v = rk[r].v;
                        if (comb_out) comb_out[posn] = comb;
                    }
                }
            }
            if (taken < quota) rc = -3;
            if (quota_out) quota_out[comb] = quota;
            if (taken_out) taken_out[comb] = taken;
            if (last_value_out) last_value_out[comb] = last_v;
            if (kth_value_out) kth_value_out[comb] = (K_m > 0) ? rk[K_m - 1].v : NAN;
        }
    }
    int64_t w = 0;
    for (int64_t t = 0; t < L; ++t)                 /* sort I in ascending order */
        if (in_I[t]) out_idx[w++] = (int32_t)t;
    if (rc == 0 && w != (int64_t)n_sink + budget) rc = -3;
    free(in_I); free(P); free(W); free(rk);
    return rc;
}


/*
 * Eq. 7: K~[t] = R(D_i) K[t] for every position t of chunk i < N_C - 1 (readings R13-R15).
 * K is bf16 [L][n_kv][d]; out is double [L][n_kv][d] (exact rotation of the bf16 values,
 * not rounded back).  Returns 0, or -1 on bad arguments.
 */
int ilre_oracle_dca_rerope(const uint16_t *K, int64_t L, int n_kv, int d, int chunk, int n_sink,
                           double theta, double *out)
{
    if (!K || !out || L < 1 || n_kv < 1 || d < 2 || (d & 1) || chunk < 1 || n_sink < 0 ||
        n_sink > L)
        return -1;
    const int half = d / 2;
    const int64_t n_chunks = (L - n_sink + chunk - 1) / chunk;                     /* R13 */
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < L; ++t) {
        int64_t i = (t < n_sink) ? 1 : 1 + (t - n_sink) / chunk;                  /* 1-based */
        const double D = (i < n_chunks - 1) ? (double)((n_chunks - 1 - i) * chunk) : 0.0; /* R14 */
        for (int g = 0; g < n_kv; ++g) {
            const uint16_t *k = K + (t * n_kv + g) * d;
            double *o = out + (t * n_kv + g) * d;
            for (int c = 0; c < half; ++c) {
                const double ang = D * pow(theta, -2.0 * (double)c / (double)d);  /* R15 */
                const double cs = cos(ang), sn = sin(ang);
                const double lo = bf16_to_double(k[c]), hi = bf16_to_double(k[c + half]);
                o[c] = lo * cs - hi * sn;
                o[c + half] = lo * sn + hi * cs;
            }
        }
    }
    return 0;
}
