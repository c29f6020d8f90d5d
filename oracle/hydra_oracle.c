/*
 * fp64 CPU oracle for the attention computation that HyDra's context-parallel engine schedules.
 *
 * THIS IS TEST INFRASTRUCTURE. It is called only by the test-suite, by the smoke check and by the
 * benchmark's cpu_baseline / reference legs. It shares no code with the CUDA library and the
 * product never routes through it.
 *
 * What it computes. The paper treats the attention kernel as a library call (Section 3.5: the
 * attention kernel dominates the layer on the pacing rank; Section 2.3 / 5.2: a packed microbatch
 * masks attention across sequence boundaries, the outer ring circulates K/V blocks and "pipelines
 * with attention as in standard ring CP").  It never prints the attention formula, so the oracle
 * is the textbook definition written out:
 *
 *   s_ij   = scale * <q_i, k_j>                      j <= i inside one packed sequence (causal)
 *   LSE_i  = ln sum_j exp(s_ij)
 *   P_ij   = exp(s_ij - LSE_i)
 *   O_i    = sum_j P_ij v_j
 *   D_i    = <dO_i, O_i>
 *   dP_ij  = <dO_i, v_j>,   dS_ij = P_ij (dP_ij - D_i)
 *   dQ_i   = scale sum_j dS_ij k_j,  dK_j = scale sum_i dS_ij q_i,  dV_j = sum_i P_ij dO_i
 *
 * A (q-chunk, kv-chunk) pair of a ring step restricts j to the pair's kv rows and emits a partial
 * (O, LSE) normalised by its own sum; the merge is LSE = ln sum_p exp(LSE_p),
 * O = sum_p exp(LSE_p - LSE) O_p.  Every loop is a plain two-pass softmax in double precision:
 * no tiling, no online rescaling, no exp2 domain, no reordering beyond "for each row".
 *
 * Inputs are bf16 bit patterns (uint16) widened exactly to double. Layouts: q,k [T,h,dqk];
 * v,dO [T,h,dv]; O, dQ, dK, dV double with the same shapes; LSE, D double [h,T].
 *
 * Parity pins (tests/test_oracle_*.py): brute-force softmax without max subtraction, closed forms
 * (L = 1, q = 0, constant k, constant v, key shift), row sums of P, gradient invariants, central
 * finite differences, torch float64 scaled_dot_product_attention + autograd, and the identity
 * "merge of the partials of any chunking == unchunked attention". The sampled forms
 * (oracle_sample_rows with its blocked gathers, oracle_sample_keys, oracle_spike_bwd) are pinned
 * against the full functions, on sequences longer than two gather blocks.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_API __attribute__((visibility("default")))

static inline double bf16_to_double(uint16_t bits)
{
    uint32_t w = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/*
 * Input element type. The method's inputs are bf16; the finite-difference pin needs steps far
 * below bf16 resolution, so the same entry points can be told that q, k, v, dO point to doubles.
 * Not thread-safe; set it, call, reset it.
 */
static int g_inputs_are_f64 = 0;
ORACLE_API void oracle_set_inputs_f64(int on) { g_inputs_are_f64 = on; }

static inline double load_in(const uint16_t *x, int64_t idx)
{
    if (g_inputs_are_f64) return ((const double *)(const void *)x)[idx];
    return bf16_to_double(x[idx]);
}

/* Gather one head of one packed sequence into a dense [len][d] double matrix. */
static double *gather_head(const uint16_t *x, int64_t tok0, int64_t len, int h, int a, int d)
{
    double *m = (double *)malloc(sizeof(double) * (size_t)(len > 0 ? len : 1) * (size_t)d);
    for (int64_t t = 0; t < len; ++t) {
        const int64_t src = ((tok0 + t) * h + a) * (int64_t)d;
        for (int e = 0; e < d; ++e) m[t * d + e] = load_in(x, src + e);
    }
    return m;
}

static inline double dot(const double *a, const double *b, int n)
{
    double s = 0.0;
    for (int e = 0; e < n; ++e) s += a[e] * b[e];
    return s;
}

/* Number of admissible keys of a pair for the query at sequence-local position p:
 * keys at positions k_start .. k_start+k_len-1 with position <= p when causal. */
static inline int64_t admissible(int64_t p, int64_t k_start, int64_t k_len, int causal)
{
    if (!causal) return k_len;
    int64_t n = p - k_start + 1;
    if (n < 0) n = 0;
    if (n > k_len) n = k_len;
    return n;
}

/*
 * One softmax row restricted to keys [k_start, k_start+nk): returns LSE (-inf if nk == 0) and
 * writes O (d_v values; zeros if nk == 0).  `sbuf` holds nk doubles of scratch.
 */
static double row_forward(const double *qi, const double *K, const double *V, int64_t k_start,
                          int64_t nk, int dqk, int dv, double scale, double *sbuf, double *o)
{
    for (int e = 0; e < dv; ++e) o[e] = 0.0;
    if (nk <= 0) return -INFINITY;
    double m = -INFINITY;
    for (int64_t j = 0; j < nk; ++j) {
        double s = scale * dot(qi, K + (k_start + j) * dqk, dqk);
        sbuf[j] = s;
        if (s > m) m = s;
    }
    double l = 0.0;
    for (int64_t j = 0; j < nk; ++j) {
        double e = exp(sbuf[j] - m);
        sbuf[j] = e;
        l += e;
    }
    for (int64_t j = 0; j < nk; ++j) {
        const double w = sbuf[j];
        const double *vj = V + (k_start + j) * dv;
        for (int e = 0; e < dv; ++e) o[e] += w * vj[e];
    }
    for (int e = 0; e < dv; ++e) o[e] /= l;
    return m + log(l);
}

/* ------------------------------------------------------------------------------------------- */
/* Unchunked forward: the definition itself.                                                    */
ORACLE_API void oracle_attn_fwd(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                                const int32_t *cu, int n_seqs, int h, int dqk, int dv, int causal,
                                double scale, double *out, double *lse)
{
    const int64_t T = cu[n_seqs];
    for (int b = 0; b < n_seqs; ++b) {
        const int64_t t0 = cu[b], L = cu[b + 1] - cu[b];
        if (L <= 0) continue;
        for (int a = 0; a < h; ++a) {
            double *Q = gather_head(q, t0, L, h, a, dqk);
            double *K = gather_head(k, t0, L, h, a, dqk);
            double *V = gather_head(v, t0, L, h, a, dv);
#pragma omp parallel
            {
                double *sbuf = (double *)malloc(sizeof(double) * (size_t)L);
#pragma omp for schedule(dynamic, 16)
                for (int64_t i = 0; i < L; ++i) {
                    int64_t nk = admissible(i, 0, L, causal);
                    double *o = out + ((t0 + i) * h + a) * (int64_t)dv;
                    lse[(int64_t)a * T + t0 + i] =
                        row_forward(Q + i * dqk, K, V, 0, nk, dqk, dv, scale, sbuf, o);
                }
                free(sbuf);
            }
            free(Q); free(K); free(V);
        }
    }
}

/* ------------------------------------------------------------------------------------------- */
/* Partial (O, LSE) of one (q-chunk, kv-chunk) pair; rows are the pair's q rows.                */
/* o_part [q_len, h, dv], lse_part [h, q_len].                                                  */
ORACLE_API void oracle_attn_partial(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                                    const int32_t *cu, int seq, int h, int dqk, int dv,
                                    int q_start, int q_len, int k_start, int k_len, int causal,
                                    double scale, double *o_part, double *lse_part)
{
    const int64_t t0 = cu[seq], L = cu[seq + 1] - cu[seq];
    if (L <= 0 || q_len <= 0) return;
    for (int a = 0; a < h; ++a) {
        double *Q = gather_head(q, t0, L, h, a, dqk);
        double *K = gather_head(k, t0, L, h, a, dqk);
        double *V = gather_head(v, t0, L, h, a, dv);
#pragma omp parallel
        {
            double *sbuf = (double *)malloc(sizeof(double) * (size_t)(k_len > 0 ? k_len : 1));
#pragma omp for schedule(dynamic, 16)
            for (int64_t r = 0; r < q_len; ++r) {
                const int64_t p = (int64_t)q_start + r;
                int64_t nk = admissible(p, k_start, k_len, causal);
                double *o = o_part + (r * h + a) * (int64_t)dv;
                lse_part[(int64_t)a * q_len + r] =
                    row_forward(Q + p * dqk, K, V, k_start, nk, dqk, dv, scale, sbuf, o);
            }
            free(sbuf);
        }
        free(Q); free(K); free(V);
    }
}

/* ------------------------------------------------------------------------------------------- */
/* n-way merge of partials that share their rows. o_parts[p] [rows,h,dv], lse_parts[p] [h,rows]. */
ORACLE_API void oracle_lse_merge(int n_parts, const double *const *o_parts,
                                 const double *const *lse_parts, int64_t rows, int h, int dv,
                                 double *out, double *lse)
{
    for (int64_t r = 0; r < rows; ++r)
        for (int a = 0; a < h; ++a) {
            double m = -INFINITY;
            for (int p = 0; p < n_parts; ++p) {
                double x = lse_parts[p][(int64_t)a * rows + r];
                if (x > m) m = x;
            }
            double *o = out + (r * h + a) * (int64_t)dv;
            for (int e = 0; e < dv; ++e) o[e] = 0.0;
            if (m == -INFINITY) { lse[(int64_t)a * rows + r] = -INFINITY; continue; }
            double z = 0.0;
            for (int p = 0; p < n_parts; ++p) z += exp(lse_parts[p][(int64_t)a * rows + r] - m);
            const double total = m + log(z);
            for (int p = 0; p < n_parts; ++p) {
                const double lp = lse_parts[p][(int64_t)a * rows + r];
                if (lp == -INFINITY) continue;
                const double w = exp(lp - total);
                const double *op = o_parts[p] + (r * h + a) * (int64_t)dv;
                for (int e = 0; e < dv; ++e) o[e] += w * op[e];
            }
            lse[(int64_t)a * rows + r] = total;
        }
}

/* ------------------------------------------------------------------------------------------- */
/* D_i = <dO_i, O_i> with the fp64 (merged) O.  d [h,T].                                        */
ORACLE_API void oracle_bwd_prep(const uint16_t *dout, const double *out, int64_t T, int h, int dv,
                                double *d)
{
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t)
        for (int a = 0; a < h; ++a) {
            double s = 0.0;
            for (int e = 0; e < dv; ++e)
                s += load_in(dout, (t * h + a) * (int64_t)dv + e) *
                     out[(t * h + a) * (int64_t)dv + e];
            d[(int64_t)a * T + t] = s;
        }
}

/* ------------------------------------------------------------------------------------------- */
/* Backward of one pair, ADDED into dq, dk, dv (double, [T,h,*]); lse and d are the merged       */
/* [h,T] arrays of the whole problem.                                                            */
ORACLE_API void oracle_attn_bwd_pair(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                                     const uint16_t *dout, const int32_t *cu, int n_seqs, int seq,
                                     int h, int dqk, int dv, int q_start, int q_len, int k_start,
                                     int k_len, int causal, double scale, const double *lse,
                                     const double *d, double *dq, double *dk, double *dvv)
{
    const int64_t T = cu[n_seqs];
    const int64_t t0 = cu[seq], L = cu[seq + 1] - cu[seq];
    if (L <= 0 || q_len <= 0 || k_len <= 0) return;
    for (int a = 0; a < h; ++a) {
        double *Q = gather_head(q, t0, L, h, a, dqk);
        double *K = gather_head(k, t0, L, h, a, dqk);
        double *V = gather_head(v, t0, L, h, a, dv);
        double *G = gather_head(dout, t0, L, h, a, dv);
        const double *lse_a = lse + (int64_t)a * T + t0;
        const double *d_a = d + (int64_t)a * T + t0;

        /* query-side pass: dQ_i */
#pragma omp parallel for schedule(dynamic, 16)
        for (int64_t r = 0; r < q_len; ++r) {
            const int64_t i = (int64_t)q_start + r;
            const int64_t nk = admissible(i, k_start, k_len, causal);
            double acc[1024];
            for (int e = 0; e < dqk; ++e) acc[e] = 0.0;
            for (int64_t jj = 0; jj < nk; ++jj) {
                const int64_t j = k_start + jj;
                const double s = scale * dot(Q + i * dqk, K + j * dqk, dqk);
                const double p = exp(s - lse_a[i]);
                const double dp = dot(G + i * dv, V + j * dv, dv);
                const double ds = p * (dp - d_a[i]);
                for (int e = 0; e < dqk; ++e) acc[e] += ds * K[j * dqk + e];
            }
            double *o = dq + ((t0 + i) * h + a) * (int64_t)dqk;
            for (int e = 0; e < dqk; ++e) o[e] += scale * acc[e];
        }

        /* key-side pass: dK_j, dV_j (scores recomputed; nothing shared between threads) */
#pragma omp parallel for schedule(dynamic, 16)
        for (int64_t jj = 0; jj < k_len; ++jj) {
            const int64_t j = (int64_t)k_start + jj;
            double acck[1024], accv[1024];
            for (int e = 0; e < dqk; ++e) acck[e] = 0.0;
            for (int e = 0; e < dv; ++e) accv[e] = 0.0;
            for (int64_t r = 0; r < q_len; ++r) {
                const int64_t i = (int64_t)q_start + r;
                if (causal && j > i) continue;
                const double s = scale * dot(Q + i * dqk, K + j * dqk, dqk);
                const double p = exp(s - lse_a[i]);
                const double dp = dot(G + i * dv, V + j * dv, dv);
                const double ds = p * (dp - d_a[i]);
                for (int e = 0; e < dqk; ++e) acck[e] += ds * Q[i * dqk + e];
                for (int e = 0; e < dv; ++e) accv[e] += p * G[i * dv + e];
            }
            double *ok = dk + ((t0 + j) * h + a) * (int64_t)dqk;
            double *ov = dvv + ((t0 + j) * h + a) * (int64_t)dv;
            for (int e = 0; e < dqk; ++e) ok[e] += scale * acck[e];
            for (int e = 0; e < dv; ++e) ov[e] += accv[e];
        }
        free(Q); free(K); free(V); free(G);
    }
}

/* ------------------------------------------------------------------------------------------- */
/* Unchunked backward: one whole-sequence pair per sequence, outputs overwritten.               */
ORACLE_API void oracle_attn_bwd(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                                const uint16_t *dout, const int32_t *cu, int n_seqs, int h,
                                int dqk, int dv, int causal, double scale, const double *out,
                                const double *lse, double *dq, double *dk, double *dvv)
{
    const int64_t T = cu[n_seqs];
    double *d = (double *)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1) * (size_t)h);
    oracle_bwd_prep(dout, out, T, h, dv, d);
    memset(dq, 0, sizeof(double) * (size_t)T * h * dqk);
    memset(dk, 0, sizeof(double) * (size_t)T * h * dqk);
    memset(dvv, 0, sizeof(double) * (size_t)T * h * dv);
    for (int b = 0; b < n_seqs; ++b) {
        const int L = cu[b + 1] - cu[b];
        oracle_attn_bwd_pair(q, k, v, dout, cu, n_seqs, b, h, dqk, dv, 0, L, 0, L, causal, scale,
                             lse, d, dq, dk, dvv);
    }
    free(d);
}

/* ------------------------------------------------------------------------------------------- */
/* One row of P (for the row-sum pin): p_row[j], j < nk, returns nk.                             */
ORACLE_API int64_t oracle_p_row(const uint16_t *q, const uint16_t *k, const int32_t *cu, int seq,
                                int h, int a, int dqk, int64_t i, int causal, double scale,
                                double *p_row)
{
    const int64_t t0 = cu[seq], L = cu[seq + 1] - cu[seq];
    double *Q = gather_head(q, t0, L, h, a, dqk);
    double *K = gather_head(k, t0, L, h, a, dqk);
    const int64_t nk = admissible(i, 0, L, causal);
    double m = -INFINITY, l = 0.0;
    for (int64_t j = 0; j < nk; ++j) {
        p_row[j] = scale * dot(Q + i * dqk, K + j * dqk, dqk);
        if (p_row[j] > m) m = p_row[j];
    }
    for (int64_t j = 0; j < nk; ++j) l += exp(p_row[j] - m);
    const double lse = m + log(l);
    for (int64_t j = 0; j < nk; ++j) p_row[j] = exp(p_row[j] - lse);
    free(Q); free(K);
    return nk;
}

/* ------------------------------------------------------------------------------------------- */
/* Sampled query rows of the unchunked problem, one head per call site loop: for each listed     */
/* (token t, head a): O (dv), LSE, D and dQ (dqk).  Cost O(i * d) per row, so the long           */
/* configurations can be checked without the full quadratic pass.                                */
ORACLE_API void oracle_sample_rows(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                                   const uint16_t *dout, const int32_t *cu, int n_seqs, int h,
                                   int dqk, int dv, int causal, double scale, int64_t n_samples,
                                   const int64_t *tok, const int32_t *head, double *o, double *lse,
                                   double *dsum, double *dq)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t s = 0; s < n_samples; ++s) {
        const int64_t t = tok[s];
        const int a = head[s];
        int b = 0;
        while (b + 1 < n_seqs && cu[b + 1] <= t) ++b;
        const int64_t t0 = cu[b], L = cu[b + 1] - cu[b], i = t - t0;
        const int64_t nk = admissible(i, 0, L, causal);
        double *qi = gather_head(q, t, 1, h, a, dqk);
        double *gi = gather_head(dout, t, 1, h, a, dv);
        /* keys and values are gathered in blocks so that a late row of a long sequence does not
         * need a private copy of the whole sequence */
        enum { BLK = 1024 };
        double *sbuf = (double *)malloc(sizeof(double) * (size_t)(nk > 0 ? nk : 1));
        double *orow = o + s * dv;
        double *dqrow = dq + s * dqk;
        for (int e = 0; e < dv; ++e) orow[e] = 0.0;
        for (int e = 0; e < dqk; ++e) dqrow[e] = 0.0;
        double m = -INFINITY, l = 0.0;
        for (int64_t j0 = 0; j0 < nk; j0 += BLK) {
            const int64_t nb = (nk - j0 < BLK) ? nk - j0 : BLK;
            double *K = gather_head(k, t0 + j0, nb, h, a, dqk);
            for (int64_t j = 0; j < nb; ++j) {
                sbuf[j0 + j] = scale * dot(qi, K + j * dqk, dqk);
                if (sbuf[j0 + j] > m) m = sbuf[j0 + j];
            }
            free(K);
        }
        for (int64_t j = 0; j < nk; ++j) l += exp(sbuf[j] - m);
        const double lse_i = (nk > 0) ? m + log(l) : -INFINITY;
        for (int64_t j0 = 0; j0 < nk; j0 += BLK) {
            const int64_t nb = (nk - j0 < BLK) ? nk - j0 : BLK;
            double *V = gather_head(v, t0 + j0, nb, h, a, dv);
            for (int64_t j = 0; j < nb; ++j) {
                const double p = exp(sbuf[j0 + j] - lse_i);
                for (int e = 0; e < dv; ++e) orow[e] += p * V[j * dv + e];
            }
            free(V);
        }
        lse[s] = lse_i;
        const double D = dot(gi, orow, dv);
        dsum[s] = D;
        for (int64_t j0 = 0; j0 < nk; j0 += BLK) {
            const int64_t nb = (nk - j0 < BLK) ? nk - j0 : BLK;
            double *K = gather_head(k, t0 + j0, nb, h, a, dqk);
            double *V = gather_head(v, t0 + j0, nb, h, a, dv);
            for (int64_t j = 0; j < nb; ++j) {
                const double p = exp(sbuf[j0 + j] - lse_i);
                const double ds = p * (dot(gi, V + j * dv, dv) - D);
                for (int e = 0; e < dqk; ++e) dqrow[e] += scale * ds * K[j * dqk + e];
            }
            free(K); free(V);
        }
        free(qi); free(gi); free(sbuf);
    }
}

/* ------------------------------------------------------------------------------------------- */
/* Sampled key rows: dK_j, dV_j for listed (token t, head a) of the unchunked problem. Each      */
/* needs every query row i >= j of its sequence (LSE_i and D_i recomputed from scratch), so      */
/* callers sample keys near the end of long sequences.                                           */
ORACLE_API void oracle_sample_keys(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                                   const uint16_t *dout, const int32_t *cu, int n_seqs, int h,
                                   int dqk, int dv, int causal, double scale, int64_t n_samples,
                                   const int64_t *tok, const int32_t *head, double *dk, double *dvv)
{
    for (int64_t s = 0; s < n_samples; ++s) {
        const int64_t t = tok[s];
        const int a = head[s];
        int b = 0;
        while (b + 1 < n_seqs && cu[b + 1] <= t) ++b;
        const int64_t t0 = cu[b], L = cu[b + 1] - cu[b], j = t - t0;
        double *Q = gather_head(q, t0, L, h, a, dqk);
        double *K = gather_head(k, t0, L, h, a, dqk);
        double *V = gather_head(v, t0, L, h, a, dv);
        double *G = gather_head(dout, t0, L, h, a, dv);
        const int64_t i_lo = causal ? j : 0;
        const int64_t n_rows = L - i_lo;
        double *acck = (double *)calloc((size_t)dqk * (size_t)n_rows, sizeof(double));
        double *accv = (double *)calloc((size_t)dv * (size_t)n_rows, sizeof(double));
#pragma omp parallel
        {
            double *sbuf = (double *)malloc(sizeof(double) * (size_t)L);
            double *orow = (double *)malloc(sizeof(double) * (size_t)dv);
#pragma omp for schedule(dynamic, 4)
            for (int64_t i = i_lo; i < L; ++i) {
                const int64_t nk = admissible(i, 0, L, causal);
                const double l = row_forward(Q + i * dqk, K, V, 0, nk, dqk, dv, scale, sbuf, orow);
                const double D = dot(G + i * dv, orow, dv);
                const double p = exp(scale * dot(Q + i * dqk, K + j * dqk, dqk) - l);
                const double ds = p * (dot(G + i * dv, V + j * dv, dv) - D);
                double *rk = acck + (i - i_lo) * dqk;
                double *rv = accv + (i - i_lo) * dv;
                for (int e = 0; e < dqk; ++e) rk[e] = scale * ds * Q[i * dqk + e];
                for (int e = 0; e < dv; ++e) rv[e] = p * G[i * dv + e];
            }
            free(sbuf); free(orow);
        }
        for (int e = 0; e < dqk; ++e) dk[s * dqk + e] = 0.0;
        for (int e = 0; e < dv; ++e) dvv[s * dv + e] = 0.0;
        for (int64_t r = 0; r < n_rows; ++r) {
            for (int e = 0; e < dqk; ++e) dk[s * dqk + e] += acck[r * dqk + e];
            for (int e = 0; e < dv; ++e) dvv[s * dv + e] += accv[r * dv + e];
        }
        free(acck); free(accv);
        free(Q); free(K); free(V); free(G);
    }
}

/* ------------------------------------------------------------------------------------------- */
/* Backward when dO is non-zero on a few query rows only ("spike" rows). dS_ij and P_ij dO_i      */
/* vanish on every other row, so dK_j and dV_j of ALL key rows, and dQ of the spike rows, follow  */
/* from one pass per spike row: two-pass softmax of the row, D_i = <dO_i, O_i>, then one loop     */
/* over the keys j <= i. Cost O(rows * L * d), which makes every key row of the long              */
/* configurations checkable element by element. The caller guarantees that dO is zero outside     */
/* the listed tokens (rows of all h heads are treated). dk [T,h,dqk], dvv [T,h,dv] are cleared    */
/* here; dq_rows is [n_rows,h,dqk].                                                               */
ORACLE_API void oracle_spike_bwd(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                                 const uint16_t *dout, const int32_t *cu, int n_seqs, int h, int dqk,
                                 int dv, int causal, double scale, int64_t n_rows, const int64_t *tok,
                                 double *dq_rows, double *dk, double *dvv)
{
    const int64_t T = cu[n_seqs];
    memset(dk, 0, sizeof(double) * (size_t)T * h * dqk);
    memset(dvv, 0, sizeof(double) * (size_t)T * h * dv);
    for (int64_t s = 0; s < n_rows; ++s) {
        const int64_t t = tok[s];
        int b = 0;
        while (b + 1 < n_seqs && cu[b + 1] <= t) ++b;
        const int64_t t0 = cu[b], L = cu[b + 1] - cu[b], i = t - t0;
        const int64_t nk = admissible(i, 0, L, causal);
        for (int a = 0; a < h; ++a) {
            double *qi = gather_head(q, t, 1, h, a, dqk);
            double *gi = gather_head(dout, t, 1, h, a, dv);
            double *sbuf = (double *)malloc(sizeof(double) * (size_t)(nk > 0 ? nk : 1));
            double *orow = (double *)calloc((size_t)dv, sizeof(double));
            double *dqrow = dq_rows + (s * h + a) * dqk;
            for (int e = 0; e < dqk; ++e) dqrow[e] = 0.0;
            /* pass 1: scores and their maximum */
            double m = -INFINITY;
#pragma omp parallel for reduction(max : m) schedule(static)
            for (int64_t j = 0; j < nk; ++j) {
                double kj[512];
                for (int e = 0; e < dqk; ++e) kj[e] = load_in(k, ((t0 + j) * h + a) * (int64_t)dqk + e);
                sbuf[j] = scale * dot(qi, kj, dqk);
                if (sbuf[j] > m) m = sbuf[j];
            }
            double l = 0.0;
            for (int64_t j = 0; j < nk; ++j) l += exp(sbuf[j] - m);
            const double lse_i = (nk > 0) ? m + log(l) : -INFINITY;
            /* pass 2: O_i, hence D_i */
            for (int64_t j = 0; j < nk; ++j) {
                const double p = exp(sbuf[j] - lse_i);
                for (int e = 0; e < dv; ++e) orow[e] += p * load_in(v, ((t0 + j) * h + a) * (int64_t)dv + e);
            }
            const double D = dot(gi, orow, dv);
            /* pass 3: every key j <= i receives this row's share; key rows are disjoint across j */
#pragma omp parallel
            {
                double *dq_priv = (double *)calloc((size_t)dqk, sizeof(double));
#pragma omp for schedule(static)
                for (int64_t j = 0; j < nk; ++j) {
                    double kj[512], vj[512];
                    for (int e = 0; e < dqk; ++e) kj[e] = load_in(k, ((t0 + j) * h + a) * (int64_t)dqk + e);
                    for (int e = 0; e < dv; ++e) vj[e] = load_in(v, ((t0 + j) * h + a) * (int64_t)dv + e);
                    const double p = exp(sbuf[j] - lse_i);
                    const double ds = p * (dot(gi, vj, dv) - D);
                    double *dkj = dk + ((t0 + j) * h + a) * (int64_t)dqk;
                    double *dvj = dvv + ((t0 + j) * h + a) * (int64_t)dv;
                    for (int e = 0; e < dqk; ++e) dkj[e] += scale * ds * qi[e];
                    for (int e = 0; e < dv; ++e) dvj[e] += p * gi[e];
                    for (int e = 0; e < dqk; ++e) dq_priv[e] += scale * ds * kj[e];
                }
#pragma omp critical
                for (int e = 0; e < dqk; ++e) dqrow[e] += dq_priv[e];
                free(dq_priv);
            }
            free(qi); free(gi); free(sbuf); free(orow);
        }
    }
}

ORACLE_API int oracle_version(void) { return 1; }
