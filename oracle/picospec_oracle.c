/*
 * CPU oracle for separate rejection sampling with sparse compression.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, double-precision
 * statement of what the hot path computes.  It shares no code, header, table
 * or constant with the CUDA path and must never be linked into or called from
 * the product library; only the tests, the smoke check and the benchmark's
 * CPU-baseline leg execute it.
 *
 * Everything is sequential and in ascending vocabulary order.  OpenMP, when
 * nthreads > 1, only distributes independent rows / sequences over threads;
 * it changes no result.
 *
 * What follows the paper (arXiv 2603.19133):
 *   - Sec. 3.3, Eq. (4): the sparse distribution is the K highest-probability
 *     components together with their vocabulary indices, stored as
 *     (int32 id, fp32 prob) pairs (8 bytes per entry; Sec. 3.3 payload figures).
 *   - Sec. 3.3: candidate i is accepted or rejected by the verifier from the
 *     probability the drafter assigned to it; at the first rejected position j
 *     the corrected token is drawn from norm(max(0, P_j(x) - Q_j(x))).
 *   - Sec. 2.1: the accept rule is the speculative-sampling one,
 *     u < min(1, p(x)/q(x)), which keeps the output law equal to the target's.
 * Where the paper is silent the reading is stated next to the code (top-p,
 * renormalisation, tie-break, temperature, bonus row, two-level inverse CDF).
 *
 *   - Sec. 3.3 read literally (pso_target_topk, pso_edge_resample): the verifier sends the K
 *     largest components of the TARGET distribution at the rejected position, unnormalised,
 *     and the edge resamples from norm(max(0, P~ - Q)) against its own dense row.
 *
 * Pins (tests/test_oracle_pins.py): library top-k + softmax closed form, sum-to-one
 * and support invariants, q~ = p special case, brute-force output law on tiny
 * vocabularies, residual-mass identity, K = 1 textbook reduction, payload sizes
 * printed in the paper.  Per-call token values on large vocabularies have no
 * printed example in the paper: "parity unpinned" against the paper for those,
 * they are pinned only through the law / invariant tests above.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define PSO_OK 0
#define PSO_EINVAL (-1)
#define PSO_ENOMEM (-2)

/* Sec. 3.3's norm(max(0, P_j - Q_j)) is undefined when max(0, P_j - Q_j) vanishes (reading: the draw
 * is then from P_j itself).  A residual whose total mass is at most this fraction of the row's
 * (which sums to one) counts as vanished: it is the resolution of double-precision sums of
 * probabilities, below which "identically zero" cannot be told from rounding. */
#define PSO_RESID_ZERO 1e-12

/* ---- helpers ------------------------------------------------------------------ */

typedef struct {
    float l; /* raw logit */
    int v;   /* vocabulary index */
} pso_key;

/* order: logit descending, then vocabulary index ascending (tie-break reading: the lower
 * index wins; the paper does not say) */
static int pso_key_cmp(const void *a, const void *b) {
    const pso_key *x = (const pso_key *)a, *y = (const pso_key *)b;
    if (x->l > y->l) return -1;
    if (x->l < y->l) return 1;
    return (x->v > y->v) - (x->v < y->v);
}

static int pso_temperature_ok(double T) { return isfinite(T) && T > 0.0; }

/* Temperature softmax of one row (Sec. 3.1 "sampling parameters"; reading: p = softmax(l / T)).
 * w[v] = exp(l[v]/T - m), Z = sum_v w[v] (ascending v).  Returns 0 if the row is usable:
 * no NaN, no +inf, at least one finite logit. */
static int pso_softmax_row(const float *l, long V, double T, double *w, double *Z_out) {
    double m = -INFINITY;
    for (long v = 0; v < V; ++v) {
        double x = (double)l[v];
        if (isnan(x) || x == INFINITY) return 1;
        x = x / T;
        if (x > m) m = x;
    }
    if (m == -INFINITY) return 1;
    double Z = 0.0;
    for (long v = 0; v < V; ++v) {
        double x = (double)l[v] / T;
        w[v] = exp(x - m);
        Z += w[v];
    }
    *Z_out = Z;
    return 0;
}

/* ---- half 1: draft-side compression -------------------------------------------- */

/* One row: Eq. (4) top-k of the temperature softmax, with the top-p cut and the
 * renormalisation the benchmark definition adds.
 *   pi      = vocabulary sorted by (logit desc, index asc)
 *   k_eff   = min(top_k > 0 ? top_k : k_max, k_max, V)
 *   top_p<1: n_p = smallest n >= 1 with sum_{j<=n} q_pi(j) >= top_p; n = min(n_p, k_eff)
 *   prob_j  = q_pi(j) / sum_{j<=n} q_pi(j), stored as fp32
 * Unused slots: idx = -1, prob = 0.  Returns n, or -1 for an unusable row. */
static int pso_compress_row(const float *l, long V, double T, int top_k, double top_p, int k_max,
                            int *idx, float *prob, double *w, pso_key *keys) {
    for (int j = 0; j < k_max; ++j) {
        idx[j] = -1;
        prob[j] = 0.0f;
    }
    double Z;
    if (!pso_temperature_ok(T) || pso_softmax_row(l, V, T, w, &Z)) return -1;
    for (long v = 0; v < V; ++v) {
        keys[v].l = l[v];
        keys[v].v = (int)v;
    }
    qsort(keys, (size_t)V, sizeof(pso_key), pso_key_cmp);

    long k_eff = top_k > 0 ? top_k : k_max;
    if (k_eff > k_max) k_eff = k_max;
    if (k_eff > V) k_eff = V;

    long n = k_eff;
    if (top_p < 1.0) {
        double cum = 0.0;
        for (long j = 0; j < k_eff; ++j) {
            cum += w[keys[j].v] / Z;
            if (cum >= top_p) {
                n = j + 1;
                break;
            }
        }
    }
    double s = 0.0;
    for (long j = 0; j < n; ++j) s += w[keys[j].v] / Z;
    for (long j = 0; j < n; ++j) {
        idx[j] = keys[j].v;
        prob[j] = (float)((w[keys[j].v] / Z) / s);
    }
    return (int)n;
}

/* Draft token x ~ q~ by inverse CDF over the n stored entries (the drafter samples its
 * candidate, Sec. 3.2 / 3.3; it has to come from the same q~ the accept test uses for the
 * output law to stay exact). */
static int pso_draw_from_sparse(const int *idx, const float *prob, int n, double u) {
    if (n <= 0) return -1;
    double total = 0.0;
    for (int j = 0; j < n; ++j) total += (double)prob[j];
    double thr = u * total, cum = 0.0;
    int last = -1;
    for (int j = 0; j < n; ++j) {
        if ((double)prob[j] > 0.0) last = j;
        cum += (double)prob[j];
        if (cum > thr) return idx[j];
    }
    return last >= 0 ? idx[last] : -1;
}

int pso_compress(const float *logits, long B, long G, long V, long row_stride,
                 const float *temperature, int top_k, float top_p, int k_max, int *q_idx,
                 float *q_prob, int *q_count, const float *u_draft, int *draft_tok,
                 int nthreads) {
    if (!logits || !temperature || !q_idx || !q_prob || !q_count) return PSO_EINVAL;
    if (B < 0 || G < 0 || V <= 0 || k_max <= 0 || row_stride < V || top_k < 0) return PSO_EINVAL;
    if (!(top_p > 0.0f)) return PSO_EINVAL;
    if ((u_draft == NULL) != (draft_tok == NULL)) return PSO_EINVAL;
    if (nthreads < 1) nthreads = 1;
    long rows = B * G;
    int err = 0;
#pragma omp parallel num_threads(nthreads)
    {
        double *w = (double *)malloc((size_t)V * sizeof(double));
        pso_key *keys = (pso_key *)malloc((size_t)V * sizeof(pso_key));
        if (!w || !keys) {
#pragma omp atomic write
            err = 1;
        }
#pragma omp barrier
        if (!err) {
#pragma omp for schedule(dynamic, 1)
            for (long r = 0; r < rows; ++r) {
                long b = r / G;
                const float *l = logits + r * row_stride;
                int *idx = q_idx + r * k_max;
                float *prob = q_prob + r * k_max;
                int n = pso_compress_row(l, V, (double)temperature[b], top_k, (double)top_p,
                                         k_max, idx, prob, w, keys);
                q_count[r] = n;
                if (draft_tok) draft_tok[r] = pso_draw_from_sparse(idx, prob, n, (double)u_draft[r]);
            }
        }
        free(w);
        free(keys);
    }
    return err ? PSO_ENOMEM : PSO_OK;
}

/* ---- residual weights and the two-level inverse CDF ------------------------------ */

/* r[v] = max(0, p[v] - q~[v]) (Sec. 3.3), with p[v] = w[v]/Z and q~ given sparsely.
 * qd is a zeroed scratch row of length V; it is zero again on return.
 * Returns R = sum_v r[v] (ascending v). */
static double pso_residual_weights(const double *w, double Z, long V, const int *idx,
                                   const float *prob, int n, double *qd, double *r) {
    for (int j = 0; j < n; ++j) qd[idx[j]] = (double)prob[j];
    double R = 0.0;
    for (long v = 0; v < V; ++v) {
        double d = w[v] / Z - qd[v];
        r[v] = d > 0.0 ? d : 0.0;
        R += r[v];
    }
    for (int j = 0; j < n; ++j) qd[idx[j]] = 0.0;
    return R;
}

/* Two-level inverse CDF over non-negative weights r[0..V) with two uniforms (reading: the
 * paper only gives the distribution; any exact sampler has the right law, this one fixes a
 * single function of (r, u1, u2)).
 *   M_c = sum of r over chunk c = [c*chunk, min((c+1)*chunk, V))
 *   c*  = first c with sum_{c'<=c} M_c' > u1 * sum_c M_c      (else the last c with M_c > 0)
 *   tok = first v in c* with sum_{v'<=v in c*} r_v' > u2 * M_c*  (else the last v with r_v > 0)
 * The strict ">" never selects a zero-weight entry.  Returns -1 if all weights are zero. */
static long pso_two_level_sample(const double *r, long V, long chunk, double u1, double u2,
                                 double *mass_out) {
    long nch = (V + chunk - 1) / chunk;
    double *M = (double *)malloc((size_t)nch * sizeof(double));
    if (!M) return -2;
    double R = 0.0;
    for (long c = 0; c < nch; ++c) {
        long v0 = c * chunk, v1 = v0 + chunk < V ? v0 + chunk : V;
        double s = 0.0;
        for (long v = v0; v < v1; ++v) s += r[v];
        M[c] = s;
        R += s;
    }
    if (mass_out) *mass_out = R;
    if (!(R > 0.0)) {
        free(M);
        return -1;
    }
    double thr1 = u1 * R, cum = 0.0;
    long cs = -1, lastc = -1;
    for (long c = 0; c < nch; ++c) {
        if (M[c] > 0.0) lastc = c;
        cum += M[c];
        if (cum > thr1) {
            cs = c;
            break;
        }
    }
    if (cs < 0) cs = lastc;
    double thr2 = u2 * M[cs];
    free(M);
    long v0 = cs * chunk, v1 = v0 + chunk < V ? v0 + chunk : V;
    long tok = -1, lastv = -1;
    cum = 0.0;
    for (long v = v0; v < v1; ++v) {
        if (r[v] > 0.0) lastv = v;
        cum += r[v];
        if (cum > thr2) {
            tok = v;
            break;
        }
    }
    return tok >= 0 ? tok : lastv;
}

/* Token from row `l` at a rejected position (residual against the sparse q~) or, when
 * use_residual == 0, from p itself (bonus row after full acceptance).  If the residual vanishes
 * (q~ >= p everywhere; total mass at most PSO_RESID_ZERO) the draw falls back to p. */
static long pso_sample_row(const float *l, long V, double T, int use_residual, const int *idx,
                           const float *prob, int n, long chunk, double u1, double u2,
                           double *w, double *qd, double *r, double *mass_out) {
    double Z;
    if (pso_softmax_row(l, V, T, w, &Z)) return -1;
    double R = 0.0;
    long tok = -1;
    if (use_residual && n > 0) {
        R = pso_residual_weights(w, Z, V, idx, prob, n, qd, r);
        if (R > PSO_RESID_ZERO) tok = pso_two_level_sample(r, V, chunk, u1, u2, &R);
    }
    if (tok < 0) {
        for (long v = 0; v < V; ++v) r[v] = w[v] / Z;
        tok = pso_two_level_sample(r, V, chunk, u1, u2, &R);
    }
    if (mass_out) *mass_out = R;
    return tok;
}

static int pso_sparse_row_ok(const int *idx, int n, int k_max, long V) {
    if (n < 0 || n > k_max) return 0;
    for (int j = 0; j < n; ++j)
        if (idx[j] < 0 || idx[j] >= V) return 0;
    return 1;
}

/* ---- half 2: target-side verification -------------------------------------------- */

/* Per sequence b (Sec. 3.3 + Sec. 2.1):
 *   for i < G: x = draft_tok[i]; qx = q~_i(x) (0 if absent); px = p_i(x);
 *              accept_i = (qx == 0) or u_i < min(1, px/qx)
 *              borderline_i = qx > 0 and |px/qx - u_i| <= 1e-6 * u_i
 *              R_i = sum_v max(0, p_i(v) - q~_i(v))
 *   a = number of leading accepts; borderline counts decisions i <= min(a, G-1)
 *   token ~ residual of row a if a < G, else ~ p of row G (bonus; Table 1 reports accepted
 *   lengths above the draft length, so a bonus token exists although Eq. (5) stops at gamma)
 * An unusable sequence (bad temperature, NaN/+inf logit, token or index out of range,
 * count outside [0, k_max]) gets accept_len = -1, token = -1, p_draft = resid_mass = -1. */
int pso_verify(const float *target_logits, long B, long G, long V, long row_stride,
               const float *temperature, const int *draft_tok, const int *q_idx,
               const float *q_prob, const int *q_count, int k_max, const float *u_accept,
               int *accept_len, double *p_draft, double *resid_mass, long long *borderline_seq,
               const float *u_resample, int *token, long chunk, int nthreads) {
    if (!target_logits || !temperature || !draft_tok || !q_idx || !q_prob || !q_count ||
        !u_accept || !accept_len || !p_draft || !resid_mass || !borderline_seq)
        return PSO_EINVAL;
    if (B < 0 || G < 0 || V <= 0 || k_max <= 0 || row_stride < V || chunk <= 0) return PSO_EINVAL;
    if ((u_resample == NULL) != (token == NULL)) return PSO_EINVAL;
    if (nthreads < 1) nthreads = 1;
    int err = 0;
#pragma omp parallel num_threads(nthreads)
    {
        double *w = (double *)malloc((size_t)V * sizeof(double));
        double *qd = (double *)calloc((size_t)V, sizeof(double));
        double *r = (double *)malloc((size_t)V * sizeof(double));
        if (!w || !qd || !r) {
#pragma omp atomic write
            err = 1;
        }
#pragma omp barrier
        if (!err) {
#pragma omp for schedule(dynamic, 1)
            for (long b = 0; b < B; ++b) {
                double T = (double)temperature[b];
                const float *rows = target_logits + b * (G + 1) * row_stride;
                int ok = pso_temperature_ok(T);
                for (long i = 0; i < G && ok; ++i) {
                    long ri = b * G + i;
                    if (draft_tok[ri] < 0 || draft_tok[ri] >= V) ok = 0;
                    if (ok && !pso_sparse_row_ok(q_idx + ri * k_max, q_count[ri], k_max, V)) ok = 0;
                }
                long a = 0;
                int still = 1;
                long long nborder = 0;
                for (long i = 0; i < G && ok; ++i) {
                    long ri = b * G + i;
                    double Z;
                    if (pso_softmax_row(rows + i * row_stride, V, T, w, &Z)) {
                        ok = 0;
                        break;
                    }
                    const int *idx = q_idx + ri * k_max;
                    const float *prob = q_prob + ri * k_max;
                    int n = q_count[ri];
                    int x = draft_tok[ri];
                    double qx = 0.0;
                    for (int j = 0; j < n; ++j)
                        if (idx[j] == x) {
                            qx = (double)prob[j];
                            break;
                        }
                    double px = w[x] / Z;
                    double u = (double)u_accept[ri];
                    int acc, border = 0;
                    if (qx > 0.0) {
                        double ratio = px / qx;
                        double lim = ratio < 1.0 ? ratio : 1.0;
                        acc = u < lim;
                        border = fabs(ratio - u) <= 1e-6 * u;
                    } else {
                        acc = 1;
                    }
                    p_draft[ri] = px;
                    resid_mass[ri] = pso_residual_weights(w, Z, V, idx, prob, n, qd, r);
                    if (still) {
                        nborder += border; /* every accepted decision and the first rejected one */
                        if (acc)
                            a += 1;
                        else
                            still = 0;
                    }
                }
                if (ok) { /* the bonus row must be usable too */
                    double Z;
                    if (pso_softmax_row(rows + G * row_stride, V, T, w, &Z)) ok = 0;
                }
                if (ok && token) {
                    long ri = b * G + a;
                    int resid = a < G;
                    long t = pso_sample_row(rows + a * row_stride, V, T, resid,
                                            resid ? q_idx + ri * k_max : NULL,
                                            resid ? q_prob + ri * k_max : NULL,
                                            resid ? q_count[ri] : 0, chunk,
                                            (double)u_resample[2 * b], (double)u_resample[2 * b + 1],
                                            w, qd, r, NULL);
                    if (t == -2) {
#pragma omp atomic write
                        err = 1;
                    }
                    token[b] = (int)t;
                }
                if (ok) {
                    accept_len[b] = (int)a;
                    borderline_seq[b] = nborder;
                } else {
                    accept_len[b] = -1;
                    borderline_seq[b] = 0;
                    if (token) token[b] = -1;
                    for (long i = 0; i < G; ++i) {
                        p_draft[b * G + i] = -1.0;
                        resid_mass[b * G + i] = -1.0;
                    }
                }
            }
        }
        free(w);
        free(qd);
        free(r);
    }
    return err ? PSO_ENOMEM : PSO_OK;
}

/* Stand-alone resampling (the edge-side local correction of Sec. 3.3): one token per
 * sequence from row pos[b] of its target logits.  pos[b] < G with a non-empty sparse row:
 * residual norm(max(0, p - q~)); pos[b] == G or an empty sparse row: p itself.
 * mass[b] = the un-normalised total the draw was taken from. */
int pso_residual_sample(const float *target_logits, long B, long G, long V, long row_stride,
                        const float *temperature, const int *pos, const int *q_idx,
                        const float *q_prob, const int *q_count, int k_max,
                        const float *u_resample, int *token, double *mass, long chunk,
                        int nthreads) {
    if (!target_logits || !temperature || !pos || !u_resample || !token) return PSO_EINVAL;
    if (B < 0 || G < 0 || V <= 0 || k_max <= 0 || row_stride < V || chunk <= 0) return PSO_EINVAL;
    if (G > 0 && (!q_idx || !q_prob || !q_count)) return PSO_EINVAL;
    if (nthreads < 1) nthreads = 1;
    int err = 0;
#pragma omp parallel num_threads(nthreads)
    {
        double *w = (double *)malloc((size_t)V * sizeof(double));
        double *qd = (double *)calloc((size_t)V, sizeof(double));
        double *r = (double *)malloc((size_t)V * sizeof(double));
        if (!w || !qd || !r) {
#pragma omp atomic write
            err = 1;
        }
#pragma omp barrier
        if (!err) {
#pragma omp for schedule(dynamic, 1)
            for (long b = 0; b < B; ++b) {
                double T = (double)temperature[b];
                long j = pos[b];
                int ok = pso_temperature_ok(T) && j >= 0 && j <= G;
                int resid = ok && j < G;
                long ri = b * G + j;
                if (resid && !pso_sparse_row_ok(q_idx + ri * k_max, q_count[ri], k_max, V)) ok = 0;
                long t = -1;
                double R = -1.0;
                if (ok) {
                    t = pso_sample_row(target_logits + (b * (G + 1) + j) * row_stride, V, T, resid,
                                       resid ? q_idx + ri * k_max : NULL,
                                       resid ? q_prob + ri * k_max : NULL,
                                       resid ? q_count[ri] : 0, chunk, (double)u_resample[2 * b],
                                       (double)u_resample[2 * b + 1], w, qd, r, &R);
                    if (t == -2) {
#pragma omp atomic write
                        err = 1;
                    }
                    if (t < 0) R = -1.0;
                }
                token[b] = (int)t;
                if (mass) mass[b] = R;
            }
        }
        free(w);
        free(qd);
        free(r);
    }
    return err ? PSO_ENOMEM : PSO_OK;
}

/* ---- prefix / incremental verification (Sec. 3.2 "Fast Verification": the verifier starts on a
 * ---- known prefix before the edge has finished its segment; Sec. 3.3: segments can be cut short) */

/* Verify the target rows [r0, r1) of every sequence that is still undecided, carrying the state
 * from the calls on earlier rows.  gamma[b] (or G when gamma is NULL) is the number of drafted
 * tokens of sequence b (latency-aware truncation makes it vary); its target rows are 0 .. gamma[b],
 * the last one being the bonus row.
 *   state_in[b] (NULL = all 1): 1 = every position before r0 was accepted, 0 = already decided
 *   (such a sequence is skipped and none of its outputs is written).
 * For an undecided sequence the positions i in [r0, min(r1, gamma)) are tested in order exactly as
 * in pso_verify.  A rejection at i decides it: accept_len = i, token from the residual of row i.
 * If all are accepted and the bonus row lies in the range (r0 <= gamma < r1): accept_len = gamma,
 * token from p at row gamma.  Otherwise it stays undecided: accept_len = -2, token = -2,
 * state_out = 1.  p_draft / resid_mass are written for the tested positions only.
 * Unusable input inside the range (or gamma outside [0, G], or gamma < r0 for an undecided
 * sequence): accept_len = -1, token = -1, state_out = 0, tested positions' p_draft / resid_mass -1.
 * Rows outside the range are never read. */
int pso_verify_range(const float *target_logits, long B, long G, long V, long row_stride,
                     const float *temperature, const int *gamma, long r0, long r1,
                     const int *state_in, const int *draft_tok, const int *q_idx,
                     const float *q_prob, const int *q_count, int k_max, const float *u_accept,
                     int *accept_len, double *p_draft, double *resid_mass, long long *borderline_seq,
                     const float *u_resample, int *token, int *state_out, long chunk, int nthreads) {
    if (!target_logits || !temperature || !accept_len || !p_draft || !resid_mass || !borderline_seq ||
        !u_resample || !token || !state_out)
        return PSO_EINVAL;
    if (G > 0 && (!draft_tok || !q_idx || !q_prob || !q_count || !u_accept)) return PSO_EINVAL;
    if (B < 0 || G < 0 || V <= 0 || k_max <= 0 || row_stride < V || chunk <= 0) return PSO_EINVAL;
    if (r0 < 0 || r1 <= r0 || r1 > G + 1) return PSO_EINVAL;
    if (nthreads < 1) nthreads = 1;
    int err = 0;
#pragma omp parallel num_threads(nthreads)
    {
        double *w = (double *)malloc((size_t)V * sizeof(double));
        double *qd = (double *)calloc((size_t)V, sizeof(double));
        double *r = (double *)malloc((size_t)V * sizeof(double));
        if (!w || !qd || !r) {
#pragma omp atomic write
            err = 1;
        }
#pragma omp barrier
        if (!err) {
#pragma omp for schedule(dynamic, 1)
            for (long b = 0; b < B; ++b) {
                borderline_seq[b] = 0;
                if (state_in && state_in[b] == 0) {
                    state_out[b] = 0;
                    continue;
                }
                double T = (double)temperature[b];
                long g = gamma ? gamma[b] : G;
                const float *rows = target_logits + b * (G + 1) * row_stride;
                int ok = pso_temperature_ok(T) && g >= 0 && g <= G && g >= r0;
                long hi = g < r1 ? g : r1; /* positions tested: [r0, hi) */
                for (long i = r0; i < hi && ok; ++i) {
                    long ri = b * G + i;
                    if (draft_tok[ri] < 0 || draft_tok[ri] >= V) ok = 0;
                    if (ok && !pso_sparse_row_ok(q_idx + ri * k_max, q_count[ri], k_max, V)) ok = 0;
                }
                long a = r0;
                int still = 1;
                long long nborder = 0;
                for (long i = r0; i < hi && ok; ++i) {
                    long ri = b * G + i;
                    double Z;
                    if (pso_softmax_row(rows + i * row_stride, V, T, w, &Z)) {
                        ok = 0;
                        break;
                    }
                    const int *idx = q_idx + ri * k_max;
                    const float *prob = q_prob + ri * k_max;
                    int n = q_count[ri];
                    int x = draft_tok[ri];
                    double qx = 0.0;
                    for (int j = 0; j < n; ++j)
                        if (idx[j] == x) {
                            qx = (double)prob[j];
                            break;
                        }
                    double px = w[x] / Z;
                    double u = (double)u_accept[ri];
                    int acc, border = 0;
                    if (qx > 0.0) {
                        double ratio = px / qx;
                        double lim = ratio < 1.0 ? ratio : 1.0;
                        acc = u < lim;
                        border = fabs(ratio - u) <= 1e-6 * u;
                    } else {
                        acc = 1;
                    }
                    p_draft[ri] = px;
                    resid_mass[ri] = pso_residual_weights(w, Z, V, idx, prob, n, qd, r);
                    if (still) {
                        nborder += border;
                        if (acc)
                            a += 1;
                        else
                            still = 0;
                    }
                }
                int rejected = ok && a < hi;
                int bonus = ok && !rejected && g < r1; /* all accepted and row g is in the range */
                if (bonus) {
                    double Z;
                    if (pso_softmax_row(rows + g * row_stride, V, T, w, &Z)) ok = 0;
                }
                if (ok && (rejected || bonus)) {
                    long ri = b * G + a;
                    long t = pso_sample_row(rows + a * row_stride, V, T, rejected,
                                            rejected ? q_idx + ri * k_max : NULL,
                                            rejected ? q_prob + ri * k_max : NULL,
                                            rejected ? q_count[ri] : 0, chunk,
                                            (double)u_resample[2 * b], (double)u_resample[2 * b + 1],
                                            w, qd, r, NULL);
                    if (t == -2) {
#pragma omp atomic write
                        err = 1;
                    }
                    token[b] = (int)t;
                    accept_len[b] = (int)a;
                    state_out[b] = 0;
                    borderline_seq[b] = nborder;
                } else if (ok) {
                    token[b] = -2;
                    accept_len[b] = -2;
                    state_out[b] = 1;
                    borderline_seq[b] = nborder;
                } else {
                    token[b] = -1;
                    accept_len[b] = -1;
                    state_out[b] = 0;
                    for (long i = r0; i < hi && i < G; ++i) {
                        p_draft[b * G + i] = -1.0;
                        resid_mass[b * G + i] = -1.0;
                    }
                }
            }
        }
        free(w);
        free(qd);
        free(r);
    }
    return err ? PSO_ENOMEM : PSO_OK;
}

/* ---- the paper's own direction (Sec. 3.3): Top-K of the target row on the verifier, ---------
 * ---- resampling against the drafter's dense row on the edge ------------------------------- */

/* Eq. (4): P_sent = the K components of the target distribution P_j with the highest
 * probabilities, with their vocabulary indices.  The probabilities are sent as they are (the
 * paper does not renormalise them).  Row j = pos[b] of sequence b's `rows_per_seq` rows.
 * Order and tie-break as everywhere: logit descending, index ascending.
 * p_count[b] = min(k, V), or -1 (ids -1, probabilities 0) for an unusable row / position. */
int pso_target_topk(const float *target_logits, long B, long rows_per_seq, long V, long row_stride,
                    const float *temperature, const int *pos, int k, int *p_idx, float *p_prob,
                    int *p_count, int nthreads) {
    if (!target_logits || !temperature || !pos || !p_idx || !p_prob || !p_count) return PSO_EINVAL;
    if (B < 0 || rows_per_seq <= 0 || V <= 0 || k <= 0 || row_stride < V) return PSO_EINVAL;
    if (nthreads < 1) nthreads = 1;
    int err = 0;
#pragma omp parallel num_threads(nthreads)
    {
        double *w = (double *)malloc((size_t)V * sizeof(double));
        pso_key *keys = (pso_key *)malloc((size_t)V * sizeof(pso_key));
        if (!w || !keys) {
#pragma omp atomic write
            err = 1;
        }
#pragma omp barrier
        if (!err) {
#pragma omp for schedule(dynamic, 1)
            for (long b = 0; b < B; ++b) {
                int *idx = p_idx + b * k;
                float *prob = p_prob + b * k;
                for (int j = 0; j < k; ++j) {
                    idx[j] = -1;
                    prob[j] = 0.0f;
                }
                p_count[b] = -1;
                long j = pos[b];
                double T = (double)temperature[b], Z;
                if (j < 0 || j >= rows_per_seq || !pso_temperature_ok(T)) continue;
                const float *l = target_logits + (b * rows_per_seq + j) * row_stride;
                if (pso_softmax_row(l, V, T, w, &Z)) continue;
                for (long v = 0; v < V; ++v) {
                    keys[v].l = l[v];
                    keys[v].v = (int)v;
                }
                qsort(keys, (size_t)V, sizeof(pso_key), pso_key_cmp);
                long n = k < V ? k : V;
                for (long t = 0; t < n; ++t) {
                    idx[t] = keys[t].v;
                    prob[t] = (float)(w[keys[t].v] / Z);
                }
                p_count[b] = (int)n;
            }
        }
        free(w);
        free(keys);
    }
    return err ? PSO_ENOMEM : PSO_OK;
}

/* Sec. 3.3, edge side: the corrected token is drawn locally from the normalised positive part
 * of P_j - Q_j.  The edge holds its own dense distribution Q_j = softmax of
 * its logits at the rejected position j = pos[b], and the K transmitted components of P_j; a
 * component that was not transmitted counts as zero, so only the K transmitted indices can carry
 * positive weight (reading: the paper does not say what the edge assumes about the rest):
 *   r_t = max(0, p_prob[t] - Q_j(p_idx[t])),  R = sum_t r_t  (stored order)
 *   token = p_idx[first t with sum_{t' <= t} r_t' > u * R], else the last t with r_t > 0
 * If R = 0 (Q_j covers every transmitted component) the draw is from the transmitted components
 * themselves, r_t = p_prob[t] (reading; the paper is silent).  mass[b] = R of the weights drawn from.
 * Unusable input (temperature, position, count or index out of range, NaN / +inf logits):
 * token = -1, mass = -1. */
int pso_edge_resample(const float *draft_logits, long B, long rows_per_seq, long V, long row_stride,
                      const float *temperature, const int *pos, const int *p_idx, const float *p_prob,
                      const int *p_count, int k, const float *u, int *token, double *mass, int nthreads) {
    if (!draft_logits || !temperature || !pos || !p_idx || !p_prob || !p_count || !u || !token) return PSO_EINVAL;
    if (B < 0 || rows_per_seq <= 0 || V <= 0 || k <= 0 || row_stride < V) return PSO_EINVAL;
    if (nthreads < 1) nthreads = 1;
    int err = 0;
#pragma omp parallel num_threads(nthreads)
    {
        double *w = (double *)malloc((size_t)V * sizeof(double));
        double *r = (double *)malloc((size_t)k * sizeof(double));
        if (!w || !r) {
#pragma omp atomic write
            err = 1;
        }
#pragma omp barrier
        if (!err) {
#pragma omp for schedule(dynamic, 1)
            for (long b = 0; b < B; ++b) {
                token[b] = -1;
                if (mass) mass[b] = -1.0;
                long j = pos[b];
                int n = p_count[b];
                double T = (double)temperature[b], Z;
                if (j < 0 || j >= rows_per_seq || n <= 0 || n > k || !pso_temperature_ok(T)) continue;
                const int *idx = p_idx + b * k;
                const float *prob = p_prob + b * k;
                int bad = 0;
                for (int t = 0; t < n; ++t)
                    if (idx[t] < 0 || idx[t] >= V) bad = 1;
                if (bad) continue;
                const float *l = draft_logits + (b * rows_per_seq + j) * row_stride;
                if (pso_softmax_row(l, V, T, w, &Z)) continue;
                double R = 0.0;
                for (int t = 0; t < n; ++t) {
                    double d = (double)prob[t] - w[idx[t]] / Z;
                    r[t] = d > 0.0 ? d : 0.0;
                    R += r[t];
                }
                if (!(R > 0.0)) {
                    R = 0.0;
                    for (int t = 0; t < n; ++t) {
                        r[t] = (double)prob[t];
                        R += r[t];
                    }
                }
                double thr = (double)u[b] * R, cum = 0.0;
                int pick = -1, last = -1;
                for (int t = 0; t < n; ++t) {
                    if (r[t] > 0.0) last = t;
                    cum += r[t];
                    if (cum > thr) {
                        pick = t;
                        break;
                    }
                }
                if (pick < 0) pick = last;
                token[b] = pick >= 0 ? idx[pick] : -1;
                if (mass) mass[b] = R;
            }
        }
        free(w);
        free(r);
    }
    return err ? PSO_ENOMEM : PSO_OK;
}
