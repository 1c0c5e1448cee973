/*
 * fp64 CPU oracle for cosine attention (Cottention, arXiv 2409.18747).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * GPU library is checked against.  It shares no code, header, table or helper
 * with the CUDA path and must never be called from it.  Only the test-suite,
 * the smoke check and the benchmark's cpu_baseline / reference arm use it.
 *
 * Notation (letters of the workload description, not the paper's):
 *   B batch, H heads, N sequence length; dk, dv the per-head sizes of keys /
 *   queries and of values / outputs (the paper's d_H_key and d_H_value of
 *   section 2.1; most workloads have dk = dv = d).
 *   q, k are contiguous row-major [B,H,N,dk] doubles, v, o, dO [B,H,N,dv];
 *   states are [B,H,dk,dv]; m is [H];
 *   s is [B] (the "sequence length" scaling base of Eq. 4, one number per
 *   batch item, >= 1).
 *
 *   x^ = x / max(||x||_2, EPS)        row normalisation, Eq. 2 / Eq. 3
 *   sigma(m) = 1/(1+exp(-m))
 *   c[b,h] = s_b ^ (-sigma(m_h))      stabilisation factor, Eq. 4
 *   v'     = c * v                    (the paper applies the factor to V)
 *
 * Every function is the paper's formula written out with no blocking, tiling
 * or re-association beyond what the cited equation itself states.  OpenMP
 * only distributes independent (b,h) pairs over host threads.
 *
 * Pins (see tests): hand-worked example, closed forms, numpy GEMM/tril
 * cross-check, finite differences, the identities between Eq. 6, 7/8 and 5;
 * the segment forms against the whole-sequence definition they compose to.
 * Readings of the paper that no printed value pins (parity unpinned by the
 * paper itself): the gradient on the clamped (||x|| <= EPS) branch, and the
 * scaling base used by a decode step.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define EPS 1e-12 /* denominator floor of the row normalisation (default of the
                     normalise routine the paper's appendix calls) */

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

static double sigmoid(double m) { return 1.0 / (1.0 + exp(-m)); }

/* Eq. 4: 1 / s^sigma(m) */
static double stab_factor(double s, double m) { return pow(s, -sigmoid(m)); }

/* Eq. 2/3: row-wise L2 normalisation; nrm[t] receives ||x_t|| (un-clamped). */
static void normalise_rows(const double* x, double* xh, double* nrm, long N, int d) {
    for (long t = 0; t < N; ++t) {
        double ss = 0.0;
        for (int a = 0; a < d; ++a) ss += x[t * d + a] * x[t * d + a];
        double n = sqrt(ss);
        double den = n > EPS ? n : EPS;
        for (int a = 0; a < d; ++a) xh[t * d + a] = x[t * d + a] / den;
        if (nrm) nrm[t] = n;
    }
}

static double dot(const double* x, const double* y, int d) {
    double acc = 0.0;
    for (int a = 0; a < d; ++a) acc += x[a] * y[a];
    return acc;
}

/* ------------------------------------------------------------------------
 * Forward, primary definition.  Eq. 3 with the factor of Eq. 4 (bidirectional)
 * and Eq. 6 with the lower-triangular mask that keeps the diagonal (causal):
 *   o_t = sum_{j in allowed(t)} (q^_t . k^_j) * c * v_j
 * --------------------------------------------------------------------- */
void oracle_fwd_quadratic(const double* q, const double* k, const double* v, const double* m,
                          const double* s, double* o, int B, int H, long N, int dk, int dv,
                          int causal) {
#pragma omp parallel for schedule(dynamic)
    for (long bh = 0; bh < (long)B * H; ++bh) {
        int b = (int)(bh / H), h = (int)(bh % H);
        const double *Q = q + bh * N * dk, *K = k + bh * N * dk, *V = v + bh * N * dv;
        double* O = o + bh * N * dv;
        double* qh = malloc(sizeof(double) * N * dk);
        double* kh = malloc(sizeof(double) * N * dk);
        double* vp = malloc(sizeof(double) * N * dv);
        normalise_rows(Q, qh, NULL, N, dk);
        normalise_rows(K, kh, NULL, N, dk);
        double c = stab_factor(s[b], m[h]);
        for (long i = 0; i < N * dv; ++i) vp[i] = V[i] * c;
        for (long t = 0; t < N; ++t) {
            for (int e = 0; e < dv; ++e) O[t * dv + e] = 0.0;
            long jend = causal ? t + 1 : N; /* mask: ones on and below the diagonal */
            for (long j = 0; j < jend; ++j) {
                double score = dot(qh + t * dk, kh + j * dk, dk);
                for (int e = 0; e < dv; ++e) O[t * dv + e] += score * vp[j * dv + e];
            }
        }
        free(qh); free(kh); free(vp);
    }
}

/* The same definition evaluated only on the listed rows (for very long N).
 * rows[r] in [0,N); out is [B,H,nrows,dv]. */
void oracle_fwd_rows(const double* q, const double* k, const double* v, const double* m,
                     const double* s, const long* rows, int nrows, double* out, int B, int H,
                     long N, int dk, int dv, int causal) {
#pragma omp parallel for schedule(dynamic) collapse(2)
    for (long bh = 0; bh < (long)B * H; ++bh) {
        for (int r = 0; r < nrows; ++r) {
            int b = (int)(bh / H), h = (int)(bh % H);
            const double *Q = q + bh * N * dk, *K = k + bh * N * dk, *V = v + bh * N * dv;
            long t = rows[r];
            double c = stab_factor(s[b], m[h]);
            double* qh = malloc(sizeof(double) * dk);
            double* kh = malloc(sizeof(double) * dk);
            normalise_rows(Q + t * dk, qh, NULL, 1, dk);
            double* O = out + (bh * nrows + r) * dv;
            for (int e = 0; e < dv; ++e) O[e] = 0.0;
            long jend = causal ? t + 1 : N;
            for (long j = 0; j < jend; ++j) {
                normalise_rows(K + j * dk, kh, NULL, 1, dk);
                double score = dot(qh, kh, dk);
                for (int e = 0; e < dv; ++e) O[e] += score * (V[j * dv + e] * c);
            }
            free(qh); free(kh);
        }
    }
}

/* ------------------------------------------------------------------------
 * Forward, recurrent form (Eq. 7 read as the recurrence of Eq. 8):
 *   S_0 = 0;  S_t = S_{t-1} + k^_t (c v_t)^T;  o_t = S_t^T q^_t.
 * The state is kept as [d_key][d_value] (the paper's H_t transposed).
 * state_out (may be NULL) receives S_N, [B,H,dk,dv].
 * --------------------------------------------------------------------- */
void oracle_fwd_recurrent(const double* q, const double* k, const double* v, const double* m,
                          const double* s, double* o, double* state_out, int B, int H, long N,
                          int dk, int dv) {
#pragma omp parallel for schedule(dynamic)
    for (long bh = 0; bh < (long)B * H; ++bh) {
        int b = (int)(bh / H), h = (int)(bh % H);
        const double *Q = q + bh * N * dk, *K = k + bh * N * dk, *V = v + bh * N * dv;
        double* O = o + bh * N * dv;
        double* S = calloc((size_t)dk * dv, sizeof(double));
        double* qh = malloc(sizeof(double) * dk);
        double* kh = malloc(sizeof(double) * dk);
        double c = stab_factor(s[b], m[h]);
        for (long t = 0; t < N; ++t) {
            normalise_rows(Q + t * dk, qh, NULL, 1, dk);
            normalise_rows(K + t * dk, kh, NULL, 1, dk);
            for (int a = 0; a < dk; ++a)
                for (int e = 0; e < dv; ++e) S[a * dv + e] += kh[a] * (V[t * dv + e] * c);
            for (int e = 0; e < dv; ++e) {
                double acc = 0.0;
                for (int a = 0; a < dk; ++a) acc += qh[a] * S[a * dv + e];
                O[t * dv + e] = acc;
            }
        }
        if (state_out) memcpy(state_out + bh * dk * dv, S, sizeof(double) * dk * dv);
        free(S); free(qh); free(kh);
    }
}

/* ------------------------------------------------------------------------
 * Bidirectional forward through the re-association of Eq. 5:
 *   S = K^^T (cV)  (dk x dv),   O = Q^ S.     state_out may be NULL.
 * --------------------------------------------------------------------- */
void oracle_fwd_bidir_assoc(const double* q, const double* k, const double* v, const double* m,
                            const double* s, double* o, double* state_out, int B, int H, long N,
                            int dk, int dv) {
#pragma omp parallel for schedule(dynamic)
    for (long bh = 0; bh < (long)B * H; ++bh) {
        int b = (int)(bh / H), h = (int)(bh % H);
        const double *Q = q + bh * N * dk, *K = k + bh * N * dk, *V = v + bh * N * dv;
        double* O = o + bh * N * dv;
        double* S = calloc((size_t)dk * dv, sizeof(double));
        double* xh = malloc(sizeof(double) * dk);
        double c = stab_factor(s[b], m[h]);
        for (long j = 0; j < N; ++j) {
            normalise_rows(K + j * dk, xh, NULL, 1, dk);
            for (int a = 0; a < dk; ++a)
                for (int e = 0; e < dv; ++e) S[a * dv + e] += xh[a] * (V[j * dv + e] * c);
        }
        for (long t = 0; t < N; ++t) {
            normalise_rows(Q + t * dk, xh, NULL, 1, dk);
            for (int e = 0; e < dv; ++e) {
                double acc = 0.0;
                for (int a = 0; a < dk; ++a) acc += xh[a] * S[a * dv + e];
                O[t * dv + e] = acc;
            }
        }
        if (state_out) memcpy(state_out + bh * dk * dv, S, sizeof(double) * dk * dv);
        free(S); free(xh);
    }
}

/* Chain rule through x^ = x / max(||x||, EPS) for one row:
 *   ||x|| > EPS : dx = (dx^ - x^ <x^, dx^>) / ||x||
 *   otherwise   : dx = dx^ / EPS        (derivative of the clamped formula) */
static void normalise_backward_row(const double* xh, double nrm, const double* dxh, double* dx,
                                   int d) {
    if (nrm > EPS) {
        double p = dot(xh, dxh, d);
        for (int a = 0; a < d; ++a) dx[a] = (dxh[a] - xh[a] * p) / nrm;
    } else {
        for (int a = 0; a < d; ++a) dx[a] = dxh[a] / EPS;
    }
}

/* Shared tail of both backward forms: from gradients w.r.t. q^, k^, v' to
 * gradients w.r.t. the raw q, k, v and the contribution of this (b,h) to dm_h.
 *   dv = c dv';   dc/dm = -ln(s) sigma(m)(1-sigma(m)) c;   dL/dc = <dv', v>. */
static double chain_to_raw(const double* qh, const double* kh, const double* nq, const double* nk,
                           const double* V, const double* dqh, const double* dkh,
                           const double* dvp, double* dQ, double* dK, double* dV, double c,
                           double s, double m, long N, int dk, int dv) {
    double dLdc = 0.0;
    for (long t = 0; t < N; ++t) {
        normalise_backward_row(qh + t * dk, nq[t], dqh + t * dk, dQ + t * dk, dk);
        normalise_backward_row(kh + t * dk, nk[t], dkh + t * dk, dK + t * dk, dk);
        for (int e = 0; e < dv; ++e) {
            dV[t * dv + e] = c * dvp[t * dv + e];
            dLdc += dvp[t * dv + e] * V[t * dv + e];
        }
    }
    double sg = sigmoid(m);
    return dLdc * (-log(s) * sg * (1.0 - sg) * c);
}

/* ------------------------------------------------------------------------
 * Backward, quadratic definition (the three gradient formulas printed after
 * Eq. 7, with dK read as (dO V'^T (.) M)^T Q^ as the appendix's cumsum code
 * implies), for L = sum(dO (.) O):
 *   G = (dO V'^T) (.) M ;  dQ^ = G K^ ;  dK^ = G^T Q^ ;  dV' = (Q^ K^^T (.) M)^T dO
 * followed by the chain rule to raw q,k,v and m.  dm is [H], overwritten.
 * --------------------------------------------------------------------- */
void oracle_bwd_quadratic(const double* q, const double* k, const double* v, const double* d_o,
                          const double* m, const double* s, double* dq, double* dk_out, double* dv_out,
                          double* dm, int B, int H, long N, int dk, int dv, int causal) {
    double* dm_bh = calloc((size_t)B * H, sizeof(double));
#pragma omp parallel for schedule(dynamic)
    for (long bh = 0; bh < (long)B * H; ++bh) {
        int b = (int)(bh / H), h = (int)(bh % H);
        const double *Q = q + bh * N * dk, *K = k + bh * N * dk, *V = v + bh * N * dv;
        const double* dO = d_o + bh * N * dv;
        size_t nk_ = (size_t)N * dk, nv_ = (size_t)N * dv;
        double *qh = malloc(sizeof(double) * nk_), *kh = malloc(sizeof(double) * nk_);
        double *vp = malloc(sizeof(double) * nv_);
        double *nq = malloc(sizeof(double) * N), *nk = malloc(sizeof(double) * N);
        double *dqh = calloc(nk_, sizeof(double)), *dkh = calloc(nk_, sizeof(double));
        double* dvp = calloc(nv_, sizeof(double));
        normalise_rows(Q, qh, nq, N, dk);
        normalise_rows(K, kh, nk, N, dk);
        double c = stab_factor(s[b], m[h]);
        for (size_t i = 0; i < nv_; ++i) vp[i] = V[i] * c;
        for (long t = 0; t < N; ++t) {
            long jend = causal ? t + 1 : N;
            for (long j = 0; j < jend; ++j) {
                double g = dot(dO + t * dv, vp + j * dv, dv);   /* G[t][j]          */
                double p = dot(qh + t * dk, kh + j * dk, dk);   /* (Q^K^^T.M)[t][j] */
                for (int a = 0; a < dk; ++a) {
                    dqh[t * dk + a] += g * kh[j * dk + a];
                    dkh[j * dk + a] += g * qh[t * dk + a];
                }
                for (int e = 0; e < dv; ++e) dvp[j * dv + e] += p * dO[t * dv + e];
            }
        }
        dm_bh[bh] = chain_to_raw(qh, kh, nq, nk, V, dqh, dkh, dvp, dq + bh * N * dk,
                                 dk_out + bh * N * dk, dv_out + bh * N * dv, c, s[b], m[h], N, dk, dv);
        free(qh); free(kh); free(vp); free(nq); free(nk); free(dqh); free(dkh); free(dvp);
    }
    for (int h = 0; h < H; ++h) {
        dm[h] = 0.0;
        for (int b = 0; b < B; ++b) dm[h] += dm_bh[(long)b * H + h];
    }
    free(dm_bh);
}

/* ------------------------------------------------------------------------
 * Causal backward in the running-sum form the paper describes: dQ^ uses the
 * forward cumulative state, dK^ and dV' use a cumulative sum that runs
 * backward in time (both sums are dk x dv):
 *   S_t = sum_{j<=t} k^_j v'_j^T ,  dq^_t = S_t do_t
 *   R_j = sum_{t>=j} q^_t do_t^T ,  dk^_j = R_j v'_j ,  dv'_j = R_j^T k^_j
 * --------------------------------------------------------------------- */
void oracle_bwd_recurrent(const double* q, const double* k, const double* v, const double* d_o,
                          const double* m, const double* s, double* dq, double* dk_out, double* dv_out,
                          double* dm, int B, int H, long N, int dk, int dv) {
    double* dm_bh = calloc((size_t)B * H, sizeof(double));
#pragma omp parallel for schedule(dynamic)
    for (long bh = 0; bh < (long)B * H; ++bh) {
        int b = (int)(bh / H), h = (int)(bh % H);
        const double *Q = q + bh * N * dk, *K = k + bh * N * dk, *V = v + bh * N * dv;
        const double* dO = d_o + bh * N * dv;
        size_t nk_ = (size_t)N * dk, nv_ = (size_t)N * dv;
        double *qh = malloc(sizeof(double) * nk_), *kh = malloc(sizeof(double) * nk_);
        double *vp = malloc(sizeof(double) * nv_);
        double *nq = malloc(sizeof(double) * N), *nk = malloc(sizeof(double) * N);
        double *dqh = malloc(sizeof(double) * nk_), *dkh = malloc(sizeof(double) * nk_);
        double* dvp = malloc(sizeof(double) * nv_);
        double* S = calloc((size_t)dk * dv, sizeof(double));
        normalise_rows(Q, qh, nq, N, dk);
        normalise_rows(K, kh, nk, N, dk);
        double c = stab_factor(s[b], m[h]);
        for (size_t i = 0; i < nv_; ++i) vp[i] = V[i] * c;
        for (long t = 0; t < N; ++t) { /* forward in time */
            for (int a = 0; a < dk; ++a)
                for (int e = 0; e < dv; ++e) S[a * dv + e] += kh[t * dk + a] * vp[t * dv + e];
            for (int a = 0; a < dk; ++a) dqh[t * dk + a] = dot(S + a * dv, dO + t * dv, dv);
        }
        memset(S, 0, sizeof(double) * dk * dv); /* now R */
        for (long j = N - 1; j >= 0; --j) { /* backward in time */
            for (int a = 0; a < dk; ++a)
                for (int e = 0; e < dv; ++e) S[a * dv + e] += qh[j * dk + a] * dO[j * dv + e];
            for (int a = 0; a < dk; ++a) dkh[j * dk + a] = dot(S + a * dv, vp + j * dv, dv);
            for (int e = 0; e < dv; ++e) {
                double acc = 0.0;
                for (int a = 0; a < dk; ++a) acc += S[a * dv + e] * kh[j * dk + a];
                dvp[j * dv + e] = acc;
            }
        }
        dm_bh[bh] = chain_to_raw(qh, kh, nq, nk, V, dqh, dkh, dvp, dq + bh * N * dk,
                                 dk_out + bh * N * dk, dv_out + bh * N * dv, c, s[b], m[h], N, dk, dv);
        free(qh); free(kh); free(vp); free(nq); free(nk); free(dqh); free(dkh); free(dvp); free(S);
    }
    for (int h = 0; h < H; ++h) {
        dm[h] = 0.0;
        for (int b = 0; b < B; ++b) dm[h] += dm_bh[(long)b * H + h];
    }
    free(dm_bh);
}

/* ------------------------------------------------------------------------
 * A segment of a longer causal sequence, forward: the recurrence of Eq. 8
 * started from a caller-held state instead of zero,
 *   S_0 = state_in;  S_t = S_{t-1} + k^_t (c v_t)^T;  o_t = S_t^T q^_t,
 * state_out = S_N (may be NULL).  The state carries the factor c of the
 * tokens it has absorbed, as the decode step's state does.
 * --------------------------------------------------------------------- */
void oracle_fwd_segment(const double* q, const double* k, const double* v, const double* m,
                        const double* s, const double* state_in, double* o, double* state_out,
                        int B, int H, long N, int dk, int dv) {
#pragma omp parallel for schedule(dynamic)
    for (long bh = 0; bh < (long)B * H; ++bh) {
        int b = (int)(bh / H), h = (int)(bh % H);
        const double *Q = q + bh * N * dk, *K = k + bh * N * dk, *V = v + bh * N * dv;
        double* O = o + bh * N * dv;
        double* S = malloc(sizeof(double) * dk * dv);
        double* qh = malloc(sizeof(double) * dk);
        double* kh = malloc(sizeof(double) * dk);
        double c = stab_factor(s[b], m[h]);
        memcpy(S, state_in + bh * dk * dv, sizeof(double) * dk * dv);
        for (long t = 0; t < N; ++t) {
            normalise_rows(Q + t * dk, qh, NULL, 1, dk);
            normalise_rows(K + t * dk, kh, NULL, 1, dk);
            for (int a = 0; a < dk; ++a)
                for (int e = 0; e < dv; ++e) S[a * dv + e] += kh[a] * (V[t * dv + e] * c);
            for (int e = 0; e < dv; ++e) {
                double acc = 0.0;
                for (int a = 0; a < dk; ++a) acc += qh[a] * S[a * dv + e];
                O[t * dv + e] = acc;
            }
        }
        if (state_out) memcpy(state_out + bh * dk * dv, S, sizeof(double) * dk * dv);
        free(S); free(qh); free(kh);
    }
}

/* ------------------------------------------------------------------------
 * Backward of such a segment, for L = sum(dO (.) O) + sum(d_state_out (.)
 * state_out), the running sums of the backward (see oracle_bwd_recurrent)
 * started from what lies outside the segment: the forward sum from state_in,
 * the reverse sum from d_state_out (the gradient that later tokens send into
 * the state this segment hands on):
 *   S_t = state_in + sum_{j<=t} k^_j v'_j^T ,           dq^_t = S_t do_t
 *   R_j = d_state_out + sum_{t>=j} q^_t do_t^T ,        dk^_j = R_j v'_j ,  dv'_j = R_j^T k^_j
 *   d_state_in = R_1
 * state_in is an input of its own (its dependence on m through earlier tokens
 * belongs to the segment that produced it), so c enters through v' = c v only
 * and the chain to raw q, k, v and m is the common one.  dm is [H], overwritten.
 * --------------------------------------------------------------------- */
void oracle_bwd_segment(const double* q, const double* k, const double* v, const double* d_o,
                        const double* state_in, const double* d_state_out, const double* m,
                        const double* s, double* dq, double* dk_out, double* dv_out,
                        double* d_state_in, double* dm, int B, int H, long N, int dk, int dv) {
    double* dm_bh = calloc((size_t)B * H, sizeof(double));
#pragma omp parallel for schedule(dynamic)
    for (long bh = 0; bh < (long)B * H; ++bh) {
        int b = (int)(bh / H), h = (int)(bh % H);
        const double *Q = q + bh * N * dk, *K = k + bh * N * dk, *V = v + bh * N * dv;
        const double* dO = d_o + bh * N * dv;
        size_t nk_ = (size_t)N * dk, nv_ = (size_t)N * dv;
        double *qh = malloc(sizeof(double) * nk_), *kh = malloc(sizeof(double) * nk_);
        double *vp = malloc(sizeof(double) * nv_);
        double *nq = malloc(sizeof(double) * N), *nk = malloc(sizeof(double) * N);
        double *dqh = malloc(sizeof(double) * nk_), *dkh = malloc(sizeof(double) * nk_);
        double* dvp = malloc(sizeof(double) * nv_);
        double* S = malloc(sizeof(double) * dk * dv);
        normalise_rows(Q, qh, nq, N, dk);
        normalise_rows(K, kh, nk, N, dk);
        double c = stab_factor(s[b], m[h]);
        for (size_t i = 0; i < nv_; ++i) vp[i] = V[i] * c;
        memcpy(S, state_in + bh * dk * dv, sizeof(double) * dk * dv);
        for (long t = 0; t < N; ++t) { /* forward in time */
            for (int a = 0; a < dk; ++a)
                for (int e = 0; e < dv; ++e) S[a * dv + e] += kh[t * dk + a] * vp[t * dv + e];
            for (int a = 0; a < dk; ++a) dqh[t * dk + a] = dot(S + a * dv, dO + t * dv, dv);
        }
        memcpy(S, d_state_out + bh * dk * dv, sizeof(double) * dk * dv); /* now R */
        for (long j = N - 1; j >= 0; --j) { /* backward in time */
            for (int a = 0; a < dk; ++a)
                for (int e = 0; e < dv; ++e) S[a * dv + e] += qh[j * dk + a] * dO[j * dv + e];
            for (int a = 0; a < dk; ++a) dkh[j * dk + a] = dot(S + a * dv, vp + j * dv, dv);
            for (int e = 0; e < dv; ++e) {
                double acc = 0.0;
                for (int a = 0; a < dk; ++a) acc += S[a * dv + e] * kh[j * dk + a];
                dvp[j * dv + e] = acc;
            }
        }
        memcpy(d_state_in + bh * dk * dv, S, sizeof(double) * dk * dv);
        dm_bh[bh] = chain_to_raw(qh, kh, nq, nk, V, dqh, dkh, dvp, dq + bh * N * dk,
                                 dk_out + bh * N * dk, dv_out + bh * N * dv, c, s[b], m[h], N, dk, dv);
        free(qh); free(kh); free(vp); free(nq); free(nk); free(dqh); free(dkh); free(dvp); free(S);
    }
    for (int h = 0; h < H; ++h) {
        dm[h] = 0.0;
        for (int b = 0; b < B; ++b) dm[h] += dm_bh[(long)b * H + h];
    }
    free(dm_bh);
}

/* ------------------------------------------------------------------------
 * One step of the recurrence of Eq. 8 on a caller-held state (in place):
 *   S <- S + k^ (c v)^T ;  o = S^T q^      (update first, then observe)
 * q,k are [B,H,dk]; v,o [B,H,dv]; state is [B,H,dk,dv]; s is [B].
 * --------------------------------------------------------------------- */
void oracle_decode_step(const double* q, const double* k, const double* v, const double* m,
                        const double* s, double* state, double* o, int B, int H, int dk, int dv) {
#pragma omp parallel for schedule(dynamic)
    for (long bh = 0; bh < (long)B * H; ++bh) {
        int b = (int)(bh / H), h = (int)(bh % H);
        double* S = state + bh * dk * dv;
        double* qh = malloc(sizeof(double) * dk);
        double* kh = malloc(sizeof(double) * dk);
        normalise_rows(q + bh * dk, qh, NULL, 1, dk);
        normalise_rows(k + bh * dk, kh, NULL, 1, dk);
        double c = stab_factor(s[b], m[h]);
        for (int a = 0; a < dk; ++a)
            for (int e = 0; e < dv; ++e) S[a * dv + e] += kh[a] * (v[bh * dv + e] * c);
        for (int e = 0; e < dv; ++e) {
            double acc = 0.0;
            for (int a = 0; a < dk; ++a) acc += qh[a] * S[a * dv + e];
            o[bh * dv + e] = acc;
        }
        free(qh); free(kh);
    }
}
