/*
 * DReSD dense-retrieval oracle: TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, brute-force CPU statement of what one DReSD draft-model call
 * computes (Algorithm 1 steps 4-7 of the paper): the query is z-scored
 * (Eq. 1), projected with the PCA matrix (Section 3.3, v_l <- v W_l),
 * scaled to unit length (Eq. 2), compared by inner product with EVERY key of
 * the datastore (Eq. 3; on unit-length vectors cosine similarity is the inner
 * product), the n most similar keys are taken, and each one's stored
 * continuation is looked up (Section 3.5, the key -> value map f_D).
 *
 * Everything floating point is done in float64, one term after another, in
 * the order the formulas are written; selection is a full sort of all N row
 * indices.  No blocking, no fusion, no early exit.  Only tests, the smoke
 * check and the benchmark's CPU-baseline leg may call this file; the CUDA
 * library shares no code, header, table or constant with it.
 *
 * Readings where the paper is silent:
 *   - epsilon of Eq. 1 and Eq. 2 are parameters (eps_z, eps_n);
 *   - Eq. 3's arg max is extended to the n best (drafts are n x L matrices,
 *     Section 5.4), ordered by score descending, ties by row index ascending;
 *   - keys are used as stored (they are unit length by construction), so the
 *     similarity is the inner product of the unit query with the stored key;
 *   - no PCA centring unless a pca_mean vector is supplied;
 *   - the value lookup copies the first draft_len stored tokens verbatim;
 *   - the first-token filter of Sections 3.1 / 3.5 (the LLM's own next token
 *     x_{t+1} rules out drafts that do not start with it) is applied BEFORE
 *     the selection: only keys whose first stored token equals first_token[b]
 *     are candidates; when fewer than n exist the tail is id -1, score
 *     -infinity, tokens -1.  first_token NULL or -1 = no filter;
 *   - Var[V] of Eq. 1 is the population variance of the sample (divide by N).
 *
 * Pins (tests/test_oracle_*.py): hand-computed cases, closed forms
 * (unit norm, scale invariance, identity keys), brute-force cross-check
 * against an independent numpy float64 formulation, and the invariants
 * self-retrieval / permutation / shard-merge.  The paper prints no worked
 * numeric example of a retrieval, so there is no paper-printed value to pin.
 */
#define _GNU_SOURCE
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORACLE_F32 = 0, ORACLE_F16 = 1, ORACLE_BF16 = 2 };

/* ---- exact decoding of stored bit patterns to float64 ------------------- */

static double decode_f16(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int expo = (h >> 10) & 0x1F;
    int mant = h & 0x3FF;
    double v;
    if (expo == 0)
        v = ldexp((double)mant, -24);               /* subnormal or zero   */
    else if (expo == 31)
        v = mant ? NAN : INFINITY;
    else
        v = ldexp(1.0 + (double)mant / 1024.0, expo - 15);
    return sign ? -v : v;
}

static double decode_bf16(uint16_t b)
{
    /* bfloat16 is the upper half of an IEEE-754 binary32. */
    int sign = (b >> 15) & 1;
    int expo = (b >> 7) & 0xFF;
    int mant = b & 0x7F;
    double v;
    if (expo == 0)
        v = ldexp((double)mant, -133);              /* 2^-126 * mant/128   */
    else if (expo == 255)
        v = mant ? NAN : INFINITY;
    else
        v = ldexp(1.0 + (double)mant / 128.0, expo - 127);
    return sign ? -v : v;
}

static double load_elem(const void *base, int64_t idx, int dtype)
{
    switch (dtype) {
    case ORACLE_F32: return (double)((const float *)base)[idx];
    case ORACLE_F16: return decode_f16(((const uint16_t *)base)[idx]);
    default:         return decode_bf16(((const uint16_t *)base)[idx]);
    }
}

double dresd_oracle_decode(uint32_t bits, int dtype)
{
    if (dtype == ORACLE_F32) {
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return dtype == ORACLE_F16 ? decode_f16((uint16_t)bits) : decode_bf16((uint16_t)bits);
}

/* ---- query preprocessing: Eq. 1 -> v W_l -> Eq. 2 ------------------------
 * queries [B][d_in] in `dtype`; mean/var/pca_mean fp32 [d_in] or NULL;
 * W [d_in][d] in `dtype` or NULL (then d must equal d_in).
 * qhat [B][d] float64 out.  Returns 0, or -1 on bad arguments.            */
int dresd_oracle_preprocess(const void *queries, int B, int d_in, int dtype,
                            const float *mean, const float *var, double eps_z,
                            const void *W, int d, const float *pca_mean,
                            double eps_n, double *qhat)
{
    if (B < 0 || d_in <= 0 || d <= 0) return -1;
    if (!W && d != d_in) return -1;
    if ((mean == NULL) != (var == NULL)) return -1;
    double *v = (double *)malloc(sizeof(double) * (size_t)d_in);
    if (!v) return -1;
    for (int b = 0; b < B; ++b) {
        for (int j = 0; j < d_in; ++j)
            v[j] = load_elem(queries, (int64_t)b * d_in + j, dtype);
        if (mean)                                              /* Eq. 1 */
            for (int j = 0; j < d_in; ++j)
                v[j] = (v[j] - (double)mean[j]) / sqrt((double)var[j] + eps_z);
        double *vl = qhat + (size_t)b * d;
        if (W) {                                               /* v_l <- v W_l */
            if (pca_mean)
                for (int j = 0; j < d_in; ++j) v[j] -= (double)pca_mean[j];
            for (int c = 0; c < d; ++c) {
                double acc = 0.0;
                for (int j = 0; j < d_in; ++j)
                    acc += v[j] * load_elem(W, (int64_t)j * d + c, dtype);
                vl[c] = acc;
            }
        } else {
            for (int c = 0; c < d; ++c) vl[c] = v[c];
        }
        double ss = 0.0;                                       /* Eq. 2 */
        for (int c = 0; c < d; ++c) ss += vl[c] * vl[c];
        double nrm = sqrt(ss);
        double den = nrm > eps_n ? nrm : eps_n;
        for (int c = 0; c < d; ++c) vl[c] /= den;
    }
    free(v);
    return 0;
}

/* ---- statistics of Eq. 1 (Section 3.2): E[V] and Var[V] per dimension -----
 * V [N][d_in] in `dtype` is the sample of full-size embeddings the statistics
 * are estimated from.  Two plain passes in float64: the mean, then the mean of
 * the squared deviations from it.  Reading: Var[V] is the population variance
 * (divide by N), as in the batch-normalisation form the equation is written in.
 * mean, var: float64 [d_in] out.  Returns 0, or -1 on bad arguments.          */
int dresd_oracle_fit_zscore(const void *V, int64_t N, int d_in, int dtype, double *mean, double *var)
{
    if (N <= 0 || d_in <= 0) return -1;
    for (int j = 0; j < d_in; ++j) {
        double s = 0.0;
        for (int64_t i = 0; i < N; ++i) s += load_elem(V, i * d_in + j, dtype);
        const double m = s / (double)N;
        double q = 0.0;
        for (int64_t i = 0; i < N; ++i) {
            const double t = load_elem(V, i * d_in + j, dtype) - m;
            q += t * t;
        }
        mean[j] = m;
        var[j] = q / (double)N;
    }
    return 0;
}

/* ---- scoring: s[i] = sum_c qhat[c] * k[i][c] for every row -------------
 * Rows are independent; `threads` > 1 only splits the row loop, the
 * arithmetic of each row is unchanged.                                      */
int dresd_oracle_scores(const void *keys, int64_t N, int d, int dtype,
                        const double *qhat, double *s, int threads)
{
    if (N < 0 || d <= 0) return -1;
    if (threads < 1) threads = 1;
#pragma omp parallel for num_threads(threads) schedule(static)
    for (int64_t i = 0; i < N; ++i) {
        double acc = 0.0;
        for (int c = 0; c < d; ++c)
            acc += qhat[c] * load_elem(keys, i * d + c, dtype);
        s[i] = acc;
    }
    return 0;
}

/* ---- ordering: score descending, then row index ascending --------------- */
static int by_score_then_id(const void *pa, const void *pb, void *ctx)
{
    const double *s = (const double *)ctx;
    int64_t a = *(const int64_t *)pa, b = *(const int64_t *)pb;
    if (s[a] > s[b]) return -1;
    if (s[a] < s[b]) return 1;
    return (a > b) - (a < b);
}

/* ---- the whole call ------------------------------------------------------
 * keys [N][d] dtype; next_tokens [N][stored_len] int32; queries [B][d_in].
 * out_ids [B][top_n] int32, out_scores [B][top_n] float64,
 * out_tokens [B][top_n][draft_len] int32; full_scores [B][N] float64 or NULL.
 * Returns 0, or -1 on bad arguments / allocation failure.                   */
int dresd_oracle_retrieve(const void *keys, const int32_t *next_tokens, int64_t N, int d,
                          int dtype, int stored_len,
                          const void *queries, int B, int d_in,
                          const float *mean, const float *var, double eps_z,
                          const void *W, const float *pca_mean, double eps_n,
                          int top_n, int draft_len, const int32_t *first_token,
                          int32_t *out_ids, double *out_scores, int32_t *out_tokens,
                          double *full_scores, int threads)
{
    if (N <= 0 || top_n < 1 || top_n > N) return -1;
    if (draft_len < 1 || draft_len > stored_len) return -1;
    if (B < 0) return -1;
    double *qhat = (double *)malloc(sizeof(double) * (size_t)(B > 0 ? B : 1) * d);
    double *s = (double *)malloc(sizeof(double) * (size_t)N);
    int64_t *order = (int64_t *)malloc(sizeof(int64_t) * (size_t)N);
    int rc = -1;
    if (!qhat || !s || !order) goto done;
    if (dresd_oracle_preprocess(queries, B, d_in, dtype, mean, var, eps_z, W, d,
                                pca_mean, eps_n, qhat) != 0)
        goto done;
    for (int b = 0; b < B; ++b) {
        dresd_oracle_scores(keys, N, d, dtype, qhat + (size_t)b * d, s, threads);
        /* candidates: every key, or (Sections 3.1, 3.5) only the keys whose stored
           continuation starts with the LLM's own next token */
        int64_t n_cand = 0;
        for (int64_t i = 0; i < N; ++i)
            if (!first_token || first_token[b] < 0 || next_tokens[i * stored_len] == first_token[b])
                order[n_cand++] = i;
        qsort_r(order, (size_t)n_cand, sizeof(int64_t), by_score_then_id, s);
        for (int r = 0; r < top_n; ++r) {
            if (r >= n_cand) {
                out_ids[(size_t)b * top_n + r] = -1;
                out_scores[(size_t)b * top_n + r] = -INFINITY;
                for (int t = 0; t < draft_len; ++t)
                    out_tokens[((size_t)b * top_n + r) * draft_len + t] = -1;
                continue;
            }
            int64_t id = order[r];
            out_ids[(size_t)b * top_n + r] = (int32_t)id;
            out_scores[(size_t)b * top_n + r] = s[id];
            for (int t = 0; t < draft_len; ++t)                 /* f_D lookup */
                out_tokens[((size_t)b * top_n + r) * draft_len + t] =
                    next_tokens[id * stored_len + t];
        }
        if (full_scores) memcpy(full_scores + (size_t)b * N, s, sizeof(double) * (size_t)N);
    }
    rc = 0;
done:
    free(qhat);
    free(s);
    free(order);
    return rc;
}

/* ---- quantised candidate search (the approximation the paper's search library makes) ----
 * The paper does not search exactly: it uses an approximate nearest-neighbour library
 * (Section 3.5), whose core device is scoring against a quantised copy of the keys.  The
 * CUDA library offers that as: 8-bit keys (E4M3: 1 sign, 4 exponent bits with bias 7, 3
 * mantissa bits, largest finite value 448, no infinities), candidates by approximate score,
 * exact re-ranking of the candidates.  Stated here step by step, exact arithmetic throughout:
 *   k8_ij = e4m3(256 k_ij)            round to nearest, ties to even, saturating at +-448
 *   h1_j  = e4m3(256 q_j),   h2_j = e4m3(16 (256 q_j - h1_j))        (two-term query)
 *   a_i   = sum_j (h1_j + h2_j / 16) k8_ij / 65536                    (approximate score)
 * The caller takes the m best a_i (ties to the lower row), scores those exactly and keeps
 * the n best.  Nothing here is printed in the paper; it is this library's definition.   */
double dresd_oracle_e4m3_decode(uint32_t code)
{
    const int sign = (code >> 7) & 1, e = (code >> 3) & 15, m = code & 7;
    double v;
    if (e == 15 && m == 7) return NAN;                       /* the only NaN pattern (and its negative) */
    if (e == 0) v = ldexp((double)m / 8.0, -6);              /* subnormal */
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return sign ? -v : v;
}

uint32_t dresd_oracle_e4m3_encode(double x)
{
    if (x != x) return 0x7F;
    const uint32_t sign = (x < 0.0 || (x == 0.0 && 1.0 / x < 0.0)) ? 0x80u : 0u;
    const double ax = fabs(x);
    /* nearest of the 127 finite non-negative values 0x00..0x7E (increasing with the code);
       a tie goes to the even code, which is the even mantissa */
    uint32_t best = 0;
    double best_err = ax;                                    /* code 0 = 0.0 */
    for (uint32_t c = 1; c <= 0x7E; ++c) {
        const double err = fabs(ax - dresd_oracle_e4m3_decode(c));
        if (err < best_err || (err == best_err && (c & 1u) == 0u)) {
            best_err = err;
            best = c;
        }
    }
    return sign | best;                                      /* values beyond 448 end at 0x7E */
}

/* approx[i] for one unit query qhat (float64 [d]) over all keys.  Returns 0 or -1.   */
int dresd_oracle_quantised_scores(const void *keys, int64_t N, int d, int dtype, const double *qhat,
                                  double *approx, int threads)
{
    if (N < 0 || d <= 0) return -1;
    double *qq = (double *)malloc(sizeof(double) * (size_t)d);
    if (!qq) return -1;
    for (int j = 0; j < d; ++j) {
        const double q256 = 256.0 * qhat[j];
        const double h1 = dresd_oracle_e4m3_decode(dresd_oracle_e4m3_encode(q256));
        const double h2 = dresd_oracle_e4m3_decode(dresd_oracle_e4m3_encode(16.0 * (q256 - h1)));
        qq[j] = h1 + h2 / 16.0;
    }
    if (threads < 1) threads = 1;
    /* 16-bit stores: the quantised value of every possible stored bit pattern, once */
    double *k8_of = NULL;
    if (dtype == ORACLE_F16 || dtype == ORACLE_BF16) {
        k8_of = (double *)malloc(sizeof(double) * 65536);
        if (!k8_of) { free(qq); return -1; }
        for (uint32_t b = 0; b < 65536; ++b) {
            const uint16_t h = (uint16_t)b;
            k8_of[b] = dresd_oracle_e4m3_decode(dresd_oracle_e4m3_encode(256.0 * load_elem(&h, 0, dtype)));
        }
    }
#pragma omp parallel for num_threads(threads) schedule(static)
    for (int64_t i = 0; i < N; ++i) {
        double acc = 0.0;
        for (int j = 0; j < d; ++j) {
            const double k8 = k8_of ? k8_of[((const uint16_t *)keys)[i * d + j]]
                                    : dresd_oracle_e4m3_decode(dresd_oracle_e4m3_encode(256.0 * load_elem(keys, i * d + j, dtype)));
            acc += qq[j] * k8;
        }
        approx[i] = acc / 65536.0;
    }
    free(k8_of);
    free(qq);
    return 0;
}

/* ---- token-level half of batch verification (Section 3.6, Fig. 3) ----------
 * prepare: tokens [B][n][L], ids [B][n] (-1 = missing neighbour).  drafts [B][n][L]:
 * after a draft's first EOS every token is EOS (the EOS id is the padding); a missing
 * neighbour is all EOS.  valid [B][n]: 0 for a missing neighbour and for a draft equal
 * to a better-ranked (lower r) present draft, else 1.                               */
int dresd_oracle_drafts_prepare(const int32_t *tokens, const int32_t *ids, int B, int n, int L,
                                int32_t eos, int32_t *drafts, int32_t *valid)
{
    if (B < 0 || n < 1 || L < 1) return -1;
    for (int b = 0; b < B; ++b)
        for (int r = 0; r < n; ++r) {
            const size_t row = ((size_t)b * n + r) * L;
            int present = ids[(size_t)b * n + r] >= 0;
            int ended = !present;
            for (int t = 0; t < L; ++t) {
                int32_t x = ended ? eos : tokens[row + t];
                drafts[row + t] = x;
                if (x == eos) ended = 1;
            }
            int ok = present;
            for (int p = 0; p < r && ok; ++p) {
                if (ids[(size_t)b * n + p] < 0) continue;
                if (memcmp(drafts + ((size_t)b * n + p) * L, drafts + row, sizeof(int32_t) * (size_t)L) == 0) ok = 0;
            }
            valid[(size_t)b * n + r] = ok;
        }
    return 0;
}

/* accept: llm [B][n][L+1] = the LLM's own token at each draft position (and after the
 * draft).  The valid draft with the longest exactly matching prefix wins (ties to the
 * lower r); out_tokens [B][L+1] = that prefix, then the LLM's token at the first
 * mismatch, then -1; out_len = prefix length + 1; out_best = -1 when no draft is valid
 * (then the single token is the LLM's own next token, llm[b][0][0]).                 */
int dresd_oracle_drafts_accept(const int32_t *drafts, const int32_t *valid, const int32_t *llm, int B, int n,
                               int L, int32_t *out_best, int32_t *out_len, int32_t *out_tokens)
{
    if (B < 0 || n < 1 || L < 1) return -1;
    for (int b = 0; b < B; ++b) {
        int best = -1, best_len = -1;
        for (int r = 0; r < n; ++r) {
            if (!valid[(size_t)b * n + r]) continue;
            int a = 0;
            while (a < L && drafts[((size_t)b * n + r) * L + a] == llm[((size_t)b * n + r) * (L + 1) + a]) ++a;
            if (a > best_len) { best_len = a; best = r; }
        }
        int len = best >= 0 ? best_len : 0;
        int src = best >= 0 ? best : 0;
        out_best[b] = best;
        out_len[b] = len + 1;
        for (int t = 0; t <= L; ++t) {
            int32_t x = -1;
            if (t < len) x = drafts[((size_t)b * n + src) * L + t];
            else if (t == len) x = llm[((size_t)b * n + src) * (L + 1) + t];
            out_tokens[(size_t)b * (L + 1) + t] = x;
        }
    }
    return 0;
}
