/*
 * tslt_oracle.c — plain CPU oracle for the TSLT hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may call this file; it shares no
 * code, header, table or constant with the CUDA library.  It is the slow, obviously
 * correct statement of what the path computes, taken step by step from the paper
 * ("Fast Collaborative Inference via Distributed Speculative Decoding"):
 *
 *   sparsify     Section 3.1 (truncated sampling: the truncation equation with its two cases
 *                the right way round, q/rho on the kept set and 0 elsewhere, as the proof of
 *                Theorem 1 uses it; the top-K and top-rho sets),
 *                Solution 1 (truncate on the logits, send only (token id, logit) pairs),
 *                Algorithm 2 / Algorithm 4 (sample x ~ Q, k times iid for multi-candidate).
 *   verify       Algorithm 3 (TokSeqVeri) with the acceptance ratio read as p/q, as in
 *                Algorithm 5 and in the proof of the multi-candidate acceptance lemma
 *                (Section 4.3), and the residual norm(max(0, P - Q)) taken over the full
 *                vocabulary.
 *   tree verify  Algorithm 5 (MCVeri, its residual update after every rejected candidate)
 *                applied at each node met on the root-to-leaf walk of Algorithm 8
 *                (TokenTreeVeri), leaf bonus token from the target row.
 *
 * All arithmetic is fp64; inputs are upcast exactly (bf16 -> fp32 -> fp64).  "Sample"
 * means inverse CDF in ascending token index driven by a supplied uniform: the first index
 * whose cumulative mass exceeds u * total.  Sorting for the truncation set is a full sort
 * by (stored logit descending, index ascending).  There is no blocking, fusion or
 * reordering: every V-wide quantity is a plain loop.
 *
 * Flags (bit set per row / sequence) mark decisions that sit within 1e-6 of a boundary;
 * a finite-precision implementation may legitimately differ there:
 *   SEL   top-p cut: a cumulative mass next to the cut is within 1e-6 of top_p
 *   SMP   draft sampling: u within 1e-6 of a CDF step next to the chosen token
 *   ACC   acceptance: u within 1e-6 of the acceptance probability (positions that matter)
 *   RES   residual / bonus sampling: u within 1e-6 (normalised) of a neighbouring CDF step
 *   DEGEN residual mass was not positive; fell back to sampling from the unmodified p
 *   EMPTY row has no finite logit
 *
 * Parity pins for every function here live in tests/test_oracle_pins.py.  What cannot be
 * pinned (agreement with the figures of the paper's experiments, which need the trained
 * models) is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_F32 0
#define ORC_BF16 1

#define FLAG_SEL 1
#define FLAG_SMP 2
#define FLAG_ACC 4
#define FLAG_RES 8
#define FLAG_DEGEN 16
#define FLAG_EMPTY 32

#define BAND 1e-6

#define ORC_OK 0
#define ORC_ERR_ARG (-1)
#define ORC_ERR_MEM (-2)

static float load_logit(const void *base, int dtype, long long i)
{
    if (dtype == ORC_F32)
        return ((const float *)base)[i];
    uint32_t bits = ((uint32_t)((const uint16_t *)base)[i]) << 16;
    float f;
    memcpy(&f, &bits, 4);
    return f;
}

static double clamp_uniform(float u)
{
    /* uniforms live in [0,1); a value >= 1 is taken as the largest float below 1 */
    if (!(u >= 0.0f))
        return 0.0;
    if (u >= 1.0f)
        return (double)nextafterf(1.0f, 0.0f);
    return (double)u;
}

/* log-sum-exp of one row at temperature T over its finite entries; returns the number of
 * finite entries.  x_v = z_v / T;  lse = m + ln sum exp(x_v - m). */
static long long row_lse(const void *row, int dtype, int V, double T, double *lse_out)
{
    double m = -INFINITY;
    long long nfinite = 0;
    for (int v = 0; v < V; ++v) {
        float z = load_logit(row, dtype, v);
        if (!isfinite(z))
            continue;
        double x = (double)z / T;
        if (x > m)
            m = x;
        ++nfinite;
    }
    if (nfinite == 0) {
        *lse_out = -INFINITY;
        return 0;
    }
    double s = 0.0;
    for (int v = 0; v < V; ++v) {
        float z = load_logit(row, dtype, v);
        if (!isfinite(z))
            continue;
        s += exp((double)z / T - m);
    }
    *lse_out = m + log(s);
    return nfinite;
}

/* probability of token v under softmax(row / T) given the row's lse */
static double row_prob(const void *row, int dtype, int v, double T, double lse)
{
    float z = load_logit(row, dtype, v);
    if (!isfinite(z) || !isfinite(lse))
        return 0.0;
    return exp((double)z / T - lse);
}

typedef struct {
    float z;
    int idx;
} ent_t;

static int cmp_ent(const void *a, const void *b)
{
    const ent_t *x = (const ent_t *)a, *y = (const ent_t *)b;
    if (x->z > y->z)
        return -1;
    if (x->z < y->z)
        return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);
}

static int cmp_int(const void *a, const void *b)
{
    int x = *(const int *)a, y = *(const int *)b;
    return (x > y) - (x < y);
}

/* Renormalised truncated distribution from the transmitted pairs (Solution 1: the verifier
 * receives logits and renormalises): q~_i = exp(l_i/T - m_S) / sum_j exp(l_j/T - m_S). */
static void rebuild_qtilde(const float *logit, int n, double T, double *qt)
{
    double m = -INFINITY;
    for (int i = 0; i < n; ++i) {
        double x = (double)logit[i] / T;
        if (isfinite(logit[i]) && x > m)
            m = x;
    }
    double W = 0.0;
    for (int i = 0; i < n; ++i) {
        qt[i] = isfinite(logit[i]) ? exp((double)logit[i] / T - m) : 0.0;
        W += qt[i];
    }
    for (int i = 0; i < n; ++i)
        qt[i] = (W > 0.0) ? qt[i] / W : 0.0;
}

/* Inverse CDF over a dense non-negative array in ascending index: first v whose cumulative
 * sum exceeds u * total; if rounding leaves none, the last v with positive mass.  Sets *near
 * when u*total is within BAND (in units of total) of the cumulative on either side. */
static int invcdf_dense(const double *w, int V, double u, int *near)
{
    double total = 0.0;
    for (int v = 0; v < V; ++v)
        total += w[v];
    *near = 0;
    if (!(total > 0.0))
        return -1;
    double target = u * total, cum = 0.0, prev = 0.0;
    int last_pos = -1, chosen = -1;
    for (int v = 0; v < V; ++v) {
        if (w[v] > 0.0)
            last_pos = v;
        prev = cum;
        cum += w[v];
        if (cum > target) {
            chosen = v;
            break;
        }
    }
    if (chosen < 0)
        return last_pos;
    /* lower step: only a decision boundary if some positive mass lies below it */
    if (prev > 0.0 && fabs(target - prev) / total < BAND)
        *near = 1;
    /* upper step: only a decision boundary if some positive mass lies above it */
    if (fabs(cum - target) / total < BAND) {
        for (int v = chosen + 1; v < V; ++v)
            if (w[v] > 0.0) {
                *near = 1;
                break;
            }
    }
    return chosen;
}

/* ------------------------------------------------------------------------------------ */
/* sparsify: Section 3.1 + Solution 1 + Algorithms 2 / 4                                 */
/* ------------------------------------------------------------------------------------ */
int tslt_oracle_sparsify(const void *logits, int dtype, int rows, int V, long long row_stride,
                         int k, double top_p, double temperature, int num_samples,
                         const float *uniforms, /* [rows, num_samples] */
                         int *idx,              /* [rows, k], pad -1 */
                         float *logit,          /* [rows, k], pad -inf */
                         int *count,            /* [rows] */
                         int *token,            /* [rows, num_samples] */
                         double *lse,           /* nullable [rows] */
                         double *mass,          /* nullable [rows] */
                         int *flags,            /* nullable [rows] */
                         double *qtilde_dense   /* nullable [rows, V] */)
{
    if (!logits || rows < 0 || V <= 0 || k <= 0 || k > V || !(temperature > 0.0) ||
        !(top_p > 0.0) || num_samples < 0 || (dtype != ORC_F32 && dtype != ORC_BF16) ||
        !idx || !logit || !count || (num_samples > 0 && (!token || !uniforms)))
        return ORC_ERR_ARG;
    size_t esz = dtype == ORC_F32 ? 4 : 2;
    ent_t *ent = (ent_t *)malloc(sizeof(ent_t) * (size_t)V);
    double *qt = (double *)malloc(sizeof(double) * (size_t)k);
    int *sel = (int *)malloc(sizeof(int) * (size_t)k);
    float *sel_logit = (float *)malloc(sizeof(float) * (size_t)k);
    if (!ent || !qt || !sel || !sel_logit) {
        free(ent); free(qt); free(sel); free(sel_logit);
        return ORC_ERR_MEM;
    }
    for (int r = 0; r < rows; ++r) {
        const void *row = (const char *)logits + (size_t)r * (size_t)row_stride * esz;
        int fl = 0;
        /* step 1: full-vocabulary softmax statistics */
        double L;
        long long nfinite = row_lse(row, dtype, V, temperature, &L);
        for (int i = 0; i < k; ++i) {
            idx[(size_t)r * k + i] = -1;
            logit[(size_t)r * k + i] = -INFINITY;
        }
        if (qtilde_dense)
            for (int v = 0; v < V; ++v)
                qtilde_dense[(size_t)r * V + v] = 0.0;
        if (nfinite == 0) {
            count[r] = 0;
            for (int s = 0; s < num_samples; ++s)
                token[(size_t)r * num_samples + s] = -1;
            if (lse) lse[r] = -INFINITY;
            if (mass) mass[r] = 0.0;
            if (flags) flags[r] = FLAG_EMPTY;
            continue;
        }
        /* step 2: order finite entries by (logit descending, index ascending) */
        int ne = 0;
        for (int v = 0; v < V; ++v) {
            float z = load_logit(row, dtype, v);
            if (isfinite(z)) {
                ent[ne].z = z;
                ent[ne].idx = v;
                ++ne;
            }
        }
        qsort(ent, (size_t)ne, sizeof(ent_t), cmp_ent);
        /* step 3: top-rho crossing n* (the crossing token is kept), then n = min(k, n*, #finite) */
        int lim = k < ne ? k : ne;
        int n;
        double c_n = 0.0;
        if (top_p >= 1.0) {
            n = lim;
            for (int i = 0; i < n; ++i)
                c_n += exp((double)ent[i].z / temperature - L);
        } else {
            double c = 0.0, c_prev = 0.0;
            n = lim;
            int crossed = 0;
            for (int i = 0; i < lim; ++i) {
                c_prev = c;
                c += exp((double)ent[i].z / temperature - L);
                if (c >= top_p) {
                    n = i + 1;
                    crossed = 1;
                    break;
                }
            }
            c_n = c;
            if (crossed) {
                /* c_{n-1} could have crossed already, or c_n could have failed to cross */
                if (n >= 2 && fabs(c_prev - top_p) < BAND)
                    fl |= FLAG_SEL;
                if (n < lim && fabs(c - top_p) < BAND)
                    fl |= FLAG_SEL;
            }
        }
        /* step 4/5: selected set in ascending index with its raw logits; renormalise */
        for (int i = 0; i < n; ++i)
            sel[i] = ent[i].idx;
        qsort(sel, (size_t)n, sizeof(int), cmp_int);
        for (int i = 0; i < n; ++i)
            sel_logit[i] = load_logit(row, dtype, sel[i]);
        rebuild_qtilde(sel_logit, n, temperature, qt);
        for (int i = 0; i < n; ++i) {
            idx[(size_t)r * k + i] = sel[i];
            logit[(size_t)r * k + i] = sel_logit[i];
            if (qtilde_dense)
                qtilde_dense[(size_t)r * V + sel[i]] = qt[i];
        }
        count[r] = n;
        if (lse) lse[r] = L;
        if (mass) mass[r] = c_n;
        /* step 6: inverse-CDF samples over the kept set in ascending index */
        for (int s = 0; s < num_samples; ++s) {
            double u = clamp_uniform(uniforms[(size_t)r * num_samples + s]);
            int near = 0;
            int pos = invcdf_dense(qt, n, u, &near);
            if (near)
                fl |= FLAG_SMP;
            token[(size_t)r * num_samples + s] = pos >= 0 ? sel[pos] : -1;
        }
        if (flags) flags[r] = fl;
    }
    free(ent); free(qt); free(sel); free(sel_logit);
    return ORC_OK;
}

/* dense target distribution p(v) = exp(z_v / T - lse) over one row */
static void dense_softmax(const void *row, int dtype, int V, double T, double lse, double *p)
{
    for (int v = 0; v < V; ++v)
        p[v] = row_prob(row, dtype, v, T, lse);
}

/* acceptance probability min(1, p/q) of Algorithm 5's test; q = 0 (token outside the
 * transmitted set, which a well-formed payload never has) accepts iff p > 0. */
static double accept_probability(double p, double q)
{
    if (q > 0.0) {
        double ratio = p / q;
        return ratio < 1.0 ? ratio : 1.0;
    }
    return p > 0.0 ? 1.0 : 0.0;
}

/* ------------------------------------------------------------------------------------ */
/* verify: Algorithm 3 (TokSeqVeri)                                                      */
/* ------------------------------------------------------------------------------------ */
int tslt_oracle_verify(const void *target_logits, int dtype, int B, int gamma, int V,
                       long long row_stride, int k,
                       const int *draft_idx,     /* [B, gamma, k] ascending, pad -1 */
                       const float *draft_logit, /* [B, gamma, k] */
                       const int *draft_count,   /* [B, gamma] */
                       const int *draft_token,   /* [B, gamma] */
                       double draft_temperature, double target_temperature,
                       const float *u_accept,    /* [B, gamma] */
                       const float *u_sample,    /* [B] */
                       int *accepted_len,        /* [B] */
                       int *out_token,           /* [B] */
                       double *accept_prob,      /* nullable [B, gamma] */
                       double *beta_hat,         /* nullable [B, gamma] */
                       double *lse_p,            /* nullable [B, gamma+1] */
                       int *flags,               /* nullable [B] */
                       double *final_dense       /* nullable [B, V]: normalised pmf sampled */)
{
    if (!target_logits || B < 0 || gamma < 0 || V <= 0 || k <= 0 || k > V ||
        !(draft_temperature > 0.0) || !(target_temperature > 0.0) ||
        (dtype != ORC_F32 && dtype != ORC_BF16) || !accepted_len || !out_token || !u_sample ||
        (gamma > 0 && (!draft_idx || !draft_logit || !draft_count || !draft_token || !u_accept)))
        return ORC_ERR_ARG;
    size_t esz = dtype == ORC_F32 ? 4 : 2;
    double *qt = (double *)malloc(sizeof(double) * (size_t)k);
    double *w = (double *)malloc(sizeof(double) * (size_t)V);
    double *L = (double *)malloc(sizeof(double) * (size_t)(gamma + 1));
    double *ap = (double *)malloc(sizeof(double) * (size_t)(gamma + 1));
    if (!qt || !w || !L || !ap) {
        free(qt); free(w); free(L); free(ap);
        return ORC_ERR_MEM;
    }
    int rc = ORC_OK;
    for (int b = 0; b < B && rc == ORC_OK; ++b) {
        int fl = 0;
        /* one parallel target pass: P_1 .. P_{gamma+1} */
        for (int j = 0; j <= gamma; ++j) {
            const void *row = (const char *)target_logits +
                              ((size_t)b * (gamma + 1) + j) * (size_t)row_stride * esz;
            row_lse(row, dtype, V, target_temperature, &L[j]);
            if (lse_p) lse_p[(size_t)b * (gamma + 1) + j] = L[j];
        }
        /* per-position acceptance probability min(1, p_j(x_j) / q~_j(x_j)) */
        for (int j = 0; j < gamma; ++j) {
            size_t dr = (size_t)b * gamma + j;
            const void *row = (const char *)target_logits +
                              ((size_t)b * (gamma + 1) + j) * (size_t)row_stride * esz;
            int n = draft_count[dr];
            if (n < 0 || n > k) { rc = ORC_ERR_ARG; break; }
            rebuild_qtilde(draft_logit + dr * k, n, draft_temperature, qt);
            int x = draft_token[dr];
            double qx = 0.0, bh = 0.0;
            for (int i = 0; i < n; ++i) {
                int v = draft_idx[dr * k + i];
                if (v < 0 || v >= V) { rc = ORC_ERR_ARG; break; }
                double pv = row_prob(row, dtype, v, target_temperature, L[j]);
                bh += pv < qt[i] ? pv : qt[i];
                if (v == x) qx = qt[i];
            }
            if (rc != ORC_OK) break;
            double px = (x >= 0 && x < V) ? row_prob(row, dtype, x, target_temperature, L[j]) : 0.0;
            ap[j] = accept_probability(px, qx);
            if (accept_prob) accept_prob[dr] = ap[j];
            if (beta_hat) beta_hat[dr] = bh;
        }
        if (rc != ORC_OK) break;
        /* the while loop: leading run of accepted positions, strict '<' */
        int a = 0;
        while (a < gamma) {
            double r = clamp_uniform(u_accept[(size_t)b * gamma + a]);
            if (fabs(r - ap[a]) < BAND)
                fl |= FLAG_ACC;
            if (r < ap[a])
                ++a;
            else
                break;
        }
        accepted_len[b] = a;
        /* correction token: residual at the rejected position, or the bonus row */
        const void *row = (const char *)target_logits +
                          ((size_t)b * (gamma + 1) + a) * (size_t)row_stride * esz;
        dense_softmax(row, dtype, V, target_temperature, L[a], w);
        if (a < gamma) {
            size_t dr = (size_t)b * gamma + a;
            int n = draft_count[dr];
            rebuild_qtilde(draft_logit + dr * k, n, draft_temperature, qt);
            double Z = 0.0;
            for (int i = 0; i < n; ++i) {
                int v = draft_idx[dr * k + i];
                double d = w[v] - qt[i];
                w[v] = d > 0.0 ? d : 0.0;
            }
            for (int v = 0; v < V; ++v)
                Z += w[v];
            if (!(Z > 0.0)) {
                fl |= FLAG_DEGEN;
                dense_softmax(row, dtype, V, target_temperature, L[a], w);
            }
        }
        int near = 0;
        double u = clamp_uniform(u_sample[b]);
        out_token[b] = invcdf_dense(w, V, u, &near);
        if (near) fl |= FLAG_RES;
        if (final_dense) {
            double tot = 0.0;
            for (int v = 0; v < V; ++v) tot += w[v];
            for (int v = 0; v < V; ++v)
                final_dense[(size_t)b * V + v] = tot > 0.0 ? w[v] / tot : 0.0;
        }
        if (flags) flags[b] = fl;
    }
    free(qt); free(w); free(L); free(ap);
    return rc;
}

/* ------------------------------------------------------------------------------------ */
/* tree verify: Algorithm 5 (MCVeri) along the walk of Algorithm 8 (TokenTreeVeri)       */
/* ------------------------------------------------------------------------------------ */
int tslt_oracle_tree_verify(const void *target_logits, int dtype, int B, int N, int V,
                            long long row_stride,
                            const int *parent,         /* [N], parent[0] = -1, parent[i] < i */
                            const int *node_draft_row, /* [N], -1 for leaves */
                            int M, int k,
                            const int *node_token,     /* [B, N] */
                            const int *draft_idx,      /* [B, M, k] */
                            const float *draft_logit,  /* [B, M, k] */
                            const int *draft_count,    /* [B, M] */
                            double draft_temperature, double target_temperature,
                            const float *u_accept,     /* [B, N] by child node */
                            const float *u_sample,     /* [B, N] by node */
                            int max_depth,
                            int *accepted_path,        /* [B, max_depth], pad -1 */
                            int *accepted_len,         /* [B] */
                            int *out_token,            /* [B] */
                            double *accept_prob,       /* nullable [B, N], NaN where untested */
                            int *flags,                /* nullable [B] */
                            double *final_dense        /* nullable [B, V] */)
{
    if (!target_logits || B < 0 || N <= 0 || V <= 0 || k <= 0 || k > V || M < 0 ||
        !(draft_temperature > 0.0) || !(target_temperature > 0.0) || !parent ||
        !node_draft_row || (dtype != ORC_F32 && dtype != ORC_BF16) || max_depth < 0 ||
        !accepted_len || !out_token || !u_sample || (max_depth > 0 && !accepted_path) ||
        (N > 1 && (!node_token || !u_accept)) ||
        (M > 0 && (!draft_idx || !draft_logit || !draft_count)))
        return ORC_ERR_ARG;
    if (parent[0] != -1)
        return ORC_ERR_ARG;
    for (int n = 1; n < N; ++n)
        if (parent[n] < 0 || parent[n] >= n)
            return ORC_ERR_ARG;
    for (int n = 0; n < N; ++n)
        if (node_draft_row[n] >= M)
            return ORC_ERR_ARG;
    size_t esz = dtype == ORC_F32 ? 4 : 2;
    double *p = (double *)malloc(sizeof(double) * (size_t)V);
    double *qd = (double *)malloc(sizeof(double) * (size_t)V);
    double *qt = (double *)malloc(sizeof(double) * (size_t)k);
    if (!p || !qd || !qt) {
        free(p); free(qd); free(qt);
        return ORC_ERR_MEM;
    }
    int rc = ORC_OK;
    for (int b = 0; b < B && rc == ORC_OK; ++b) {
        int fl = 0, len = 0, node = 0;
        for (int d = 0; d < max_depth; ++d)
            accepted_path[(size_t)b * max_depth + d] = -1;
        if (accept_prob)
            for (int n = 0; n < N; ++n)
                accept_prob[(size_t)b * N + n] = NAN;
        for (;;) {
            const void *row = (const char *)target_logits +
                              ((size_t)b * N + node) * (size_t)row_stride * esz;
            double L;
            row_lse(row, dtype, V, target_temperature, &L);
            dense_softmax(row, dtype, V, target_temperature, L, p); /* p^(1) = P_node */
            int dr = node_draft_row[node];
            int accepted = 0;
            if (dr >= 0) {
                size_t dro = (size_t)b * M + dr;
                int n = draft_count[dro];
                if (n < 0 || n > k) { rc = ORC_ERR_ARG; break; }
                rebuild_qtilde(draft_logit + dro * k, n, draft_temperature, qt);
                for (int v = 0; v < V; ++v) qd[v] = 0.0;
                for (int i = 0; i < n; ++i) {
                    int v = draft_idx[dro * k + i];
                    if (v < 0 || v >= V) { rc = ORC_ERR_ARG; break; }
                    qd[v] = qt[i];
                }
                if (rc != ORC_OK) break;
                /* candidates x^(1..k) = children in ascending node id */
                for (int c = node + 1; c < N; ++c) {
                    if (parent[c] != node) continue;
                    int x = node_token[(size_t)b * N + c];
                    double px = (x >= 0 && x < V) ? p[x] : 0.0;
                    double qx = (x >= 0 && x < V) ? qd[x] : 0.0;
                    double a = accept_probability(px, qx);
                    if (accept_prob) accept_prob[(size_t)b * N + c] = a;
                    double r = clamp_uniform(u_accept[(size_t)b * N + c]);
                    if (fabs(r - a) < BAND) fl |= FLAG_ACC;
                    if (r < a) {
                        if (len >= max_depth) { rc = ORC_ERR_ARG; break; }
                        accepted_path[(size_t)b * max_depth + len] = c;
                        ++len;
                        node = c;
                        accepted = 1;
                        break;
                    }
                    /* rejected: p^(i+1) = norm(max(0, p^(i) - q~)) over the full vocabulary */
                    double Z = 0.0;
                    for (int v = 0; v < V; ++v) {
                        double d = p[v] - qd[v];
                        Z += d > 0.0 ? d : 0.0;
                    }
                    if (Z > 0.0) {
                        for (int v = 0; v < V; ++v) {
                            double d = p[v] - qd[v];
                            p[v] = d > 0.0 ? d / Z : 0.0;
                        }
                    } else {
                        fl |= FLAG_DEGEN;
                    }
                }
                if (rc != ORC_OK) break;
            }
            if (accepted)
                continue;
            /* leaf: bonus token from the target row; internal: sample p^(k+1) */
            int near = 0;
            double u = clamp_uniform(u_sample[(size_t)b * N + node]);
            out_token[b] = invcdf_dense(p, V, u, &near);
            if (near) fl |= FLAG_RES;
            if (final_dense) {
                double tot = 0.0;
                for (int v = 0; v < V; ++v) tot += p[v];
                for (int v = 0; v < V; ++v)
                    final_dense[(size_t)b * V + v] = tot > 0.0 ? p[v] / tot : 0.0;
            }
            break;
        }
        accepted_len[b] = len;
        if (flags) flags[b] = fl;
    }
    free(p); free(qd); free(qt);
    return rc;
}
