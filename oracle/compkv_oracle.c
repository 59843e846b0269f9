/*
 * CompKV CPU oracle -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * A plain, slow, double-precision restatement of what the decode path computes,
 * written from the paper's equations: straight loops, no blocking, no fusion, no
 * reordering beyond what each equation states.  Only tests, the smoke check and
 * the bench's CPU-baseline leg may call it.  It shares no code with the CUDA
 * library and neither includes the other.
 *
 * One call handles one "unit": one KV head of one sequence together with the G
 * query heads that share it (Sec. 3.1).  Inputs are float32 arrays holding the
 * bf16-rounded values both sides consume; all arithmetic and outputs are double.
 *
 * Notation follows the paper: d head dimension, N tokens, blocks b of |b| tokens
 * cut from token 0 in fixed size bs (the last one may be partial), X = ceil(N/bs),
 * z_{g,j} = q_g . k_j * scale, zbar_{g,b} the block-mean logit, Z_{g,b} = sum_j e^{z_{g,j}}.
 *
 * Pins (tests/test_oracle_pins.py): dense vs a library attention routine; select-all
 * and size-1 / constant-key blocks reproduce dense (Eq. 12, Eq. 1); KL by its
 * definition vs the log-partition gap (Eq. 4); Drop ordering (App. A.5); the
 * second-order expansions (App. A.2); variance identities (App. A.4); brute-force
 * top-k and brute-force subset search (Eq. 2, Eq. 11); the paper's printed counts.
 * Parity unpinned (fixed by a stated reading only): the RoPE pair layout behind the
 * coordinate groups, and tie order beyond "stable".
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

/* Coordinate group of coordinate i (App. A.4): r equal consecutive groups of RoPE
 * frequency pairs, both coordinates of a pair in the same group; r == d means one
 * coordinate per group.  layout 0: pair p = (2p, 2p+1), i.e. groups are contiguous
 * coordinate ranges.  layout 1: pair p = (p, p + d/2). */
int ckvo_group_of(int i, int d, int r, int layout)
{
    if (r == d) return i;
    if (layout == 0) return i / (d / r);
    int half = d / 2;
    int p = i < half ? i : i - half;
    return p / (half / r);
}

static double dotf(const float *a, const float *b, int d)
{
    double s = 0.0;
    for (int i = 0; i < d; ++i) s += (double)a[i] * (double)b[i];
    return s;
}

/* Dense softmax attention of G query heads over N tokens (Sec. 3.1; Eq. 12 with S = all blocks).
 * out [G][d], lse [G] = log sum_j e^{z_{g,j}}. */
void ckvo_dense(const float *q, const float *K, const float *V, int N, int G, int d, double scale,
                double *out, double *lse)
{
    double *z = (double *)malloc(sizeof(double) * (size_t)N);
    for (int g = 0; g < G; ++g) {
        double m = -INFINITY;
        for (int j = 0; j < N; ++j) {
            z[j] = dotf(q + (size_t)g * d, K + (size_t)j * d, d) * scale;
            if (z[j] > m) m = z[j];
        }
        double den = 0.0;
        for (int i = 0; i < d; ++i) out[(size_t)g * d + i] = 0.0;
        for (int j = 0; j < N; ++j) {
            double w = exp(z[j] - m);
            den += w;
            for (int i = 0; i < d; ++i) out[(size_t)g * d + i] += w * (double)V[(size_t)j * d + i];
        }
        for (int i = 0; i < d; ++i) out[(size_t)g * d + i] /= den;
        lse[g] = m + log(den);
    }
    free(z);
}

/* Block summaries (Sec. 4.2: {|b|, kbar_b, Dbar_b, vbar_b}; Eq. 8 right half).
 * Blocks [first_block, first_block + nblocks) of a cache of N tokens.
 * cnt [nblocks], kmean [nblocks][d], Dbar [nblocks][r], vmean [nblocks][d].
 * Dbar_t = 1/(|b| |G_t|) sum_j sum_{i in G_t} (k_{j,i} - kbar_{b,i})^2  (population variance). */
void ckvo_stats(const float *K, const float *V, int N, int d, int bs, int r, int layout,
                int first_block, int nblocks, int *cnt, double *kmean, double *Dbar, double *vmean)
{
    for (int bb = 0; bb < nblocks; ++bb) {
        int b = first_block + bb;
        int lo = b * bs;
        int hi = lo + bs < N ? lo + bs : N;
        int n = hi - lo;
        cnt[bb] = n;
        double *km = kmean + (size_t)bb * d, *vm = vmean + (size_t)bb * d, *D = Dbar + (size_t)bb * r;
        for (int i = 0; i < d; ++i) {
            double sk = 0.0, sv = 0.0;
            for (int j = lo; j < hi; ++j) {
                sk += (double)K[(size_t)j * d + i];
                sv += (double)V[(size_t)j * d + i];
            }
            km[i] = sk / n;
            vm[i] = sv / n;
        }
        for (int t = 0; t < r; ++t) D[t] = 0.0;
        int gsize = d / r;
        for (int i = 0; i < d; ++i) {
            double ss = 0.0;
            for (int j = lo; j < hi; ++j) {
                double dv = (double)K[(size_t)j * d + i] - km[i];
                ss += dv * dv;
            }
            D[ckvo_group_of(i, d, r, layout)] += ss;
        }
        for (int t = 0; t < r; ++t) D[t] /= ((double)n * (double)gsize);
    }
}

/* Scorer (Eq. 8 left half, Eq. 9, Eq. 10).  All outputs [G][X] except S [X].
 * sigma2_{g,b} = scale^2 sum_t (sum_{i in G_t} q_{g,i}^2) Dbar_{b,t}
 *                (Eq. 8 prints 1/d: App. A.4 obtains it from z - zbar = q (k - kbar)^T / sqrt(d), i.e. it is the
 *                 squared logit scale, which is 1/d for the default scale)
 * zbar_{g,b}   = q_g . kbar_b * scale
 * phat_{g,b}   = |b| exp(zbar + sigma2/2) / sum_c |c| exp(zbar_c + sigma2_c/2)   (over all blocks)
 * S_b          = sum_g phat_{g,b} sigma2_{g,b}.
 * mass_order: 2 = Eq. 9 as printed; 1 = the first-order mass of the paper's ablation (no sigma2/2 term).
 * outer_var:  1 = Eq. 10 as printed; 0 = estimated-mass ranking (no outer variance factor). */
void ckvo_scores(const float *q, const int *cnt, const double *kmean, const double *Dbar, int X, int G,
                 int d, int r, int layout, double scale, int mass_order, int outer_var,
                 double *zbar, double *sigma2, double *phat, double *S)
{
    double *w = (double *)malloc(sizeof(double) * (size_t)r);
    for (int b = 0; b < X; ++b) S[b] = 0.0;
    for (int g = 0; g < G; ++g) {
        const float *qg = q + (size_t)g * d;
        for (int t = 0; t < r; ++t) w[t] = 0.0;
        for (int i = 0; i < d; ++i) w[ckvo_group_of(i, d, r, layout)] += (double)qg[i] * (double)qg[i];
        double *zb = zbar + (size_t)g * X, *s2 = sigma2 + (size_t)g * X, *ph = phat + (size_t)g * X;
        double m = -INFINITY;
        for (int b = 0; b < X; ++b) {
            double acc = 0.0;
            for (int i = 0; i < d; ++i) acc += (double)qg[i] * kmean[(size_t)b * d + i];
            zb[b] = acc * scale;
            double v = 0.0;
            for (int t = 0; t < r; ++t) v += w[t] * Dbar[(size_t)b * r + t];
            s2[b] = v * scale * scale;
            double l = log((double)cnt[b]) + zb[b] + (mass_order == 2 ? 0.5 * s2[b] : 0.0);
            ph[b] = l;
            if (l > m) m = l;
        }
        double den = 0.0;
        for (int b = 0; b < X; ++b) {
            ph[b] = exp(ph[b] - m);
            den += ph[b];
        }
        for (int b = 0; b < X; ++b) {
            ph[b] /= den;
            S[b] += ph[b] * (outer_var ? s2[b] : 1.0);
        }
    }
    free(w);
}

/* Selection (Eq. 11): mandatory set F = first `sink` blocks and last `recent` blocks (overlap
 * counted once), plus the K - |F| highest-scoring other blocks; equal scores go to the lower
 * block id ("stable"); ids returned ascending.  K >= X selects every block.
 * Returns |S|, or -1 when K < |F| (budget too small). */
typedef struct { double s; int b; } ckvo_cand;

static int cand_cmp(const void *a, const void *b)
{
    const ckvo_cand *x = (const ckvo_cand *)a, *y = (const ckvo_cand *)b;
    if (x->s > y->s) return -1;
    if (x->s < y->s) return 1;
    return x->b - y->b;
}

int ckvo_select(const double *S, int X, int K, int sink, int recent, int *ids)
{
    if (K >= X) {
        for (int b = 0; b < X; ++b) ids[b] = b;
        return X;
    }
    char *in = (char *)calloc((size_t)X, 1);
    int nf = 0;
    for (int b = 0; b < X; ++b)
        if (b < sink || b >= X - recent) { in[b] = 1; ++nf; }
    if (K < nf) { free(in); return -1; }
    ckvo_cand *c = (ckvo_cand *)malloc(sizeof(ckvo_cand) * (size_t)X);
    int nc = 0;
    for (int b = 0; b < X; ++b)
        if (!in[b]) { c[nc].s = S[b]; c[nc].b = b; ++nc; }
    qsort(c, (size_t)nc, sizeof(ckvo_cand), cand_cmp);
    for (int i = 0; i < K - nf; ++i) in[c[i].b] = 1;
    int n = 0;
    for (int b = 0; b < X; ++b)
        if (in[b]) ids[n++] = b;
    free(c);
    free(in);
    return n;
}

/* Compensated sparse attention (Eq. 12): selected blocks contribute their tokens exactly,
 * every other block contributes |b| e^{zbar_{g,b}} with value vbar_b, one shared normaliser.
 * zbar is computed from the stored mean key.  drop != 0 leaves the unselected blocks out
 * altogether (the uncompensated variant of App. A.5).
 * ids ascending, nsel of them.  out [G][d]; lse [G] = log of the shared normaliser. */
void ckvo_sparse(const float *q, const float *K, const float *V, int N, int G, int d, int bs,
                 const int *cnt, const double *kmean, const double *vmean, const int *ids, int nsel,
                 double scale, int drop, double *out, double *lse)
{
    int X = (N + bs - 1) / bs;
    char *sel = (char *)calloc((size_t)X, 1);
    for (int i = 0; i < nsel; ++i) sel[ids[i]] = 1;
    double *zt = (double *)malloc(sizeof(double) * (size_t)N);
    double *zb = (double *)malloc(sizeof(double) * (size_t)X);
    for (int g = 0; g < G; ++g) {
        const float *qg = q + (size_t)g * d;
        double m = -INFINITY;
        for (int b = 0; b < X; ++b) {
            if (sel[b]) {
                int lo = b * bs, hi = lo + bs < N ? lo + bs : N;
                for (int j = lo; j < hi; ++j) {
                    zt[j] = dotf(qg, K + (size_t)j * d, d) * scale;
                    if (zt[j] > m) m = zt[j];
                }
            } else if (!drop) {
                double acc = 0.0;
                for (int i = 0; i < d; ++i) acc += (double)qg[i] * kmean[(size_t)b * d + i];
                zb[b] = acc * scale;
                if (zb[b] > m) m = zb[b];
            }
        }
        double den = 0.0;
        double *o = out + (size_t)g * d;
        for (int i = 0; i < d; ++i) o[i] = 0.0;
        for (int b = 0; b < X; ++b) {
            if (sel[b]) {
                int lo = b * bs, hi = lo + bs < N ? lo + bs : N;
                for (int j = lo; j < hi; ++j) {
                    double w = exp(zt[j] - m);
                    den += w;
                    for (int i = 0; i < d; ++i) o[i] += w * (double)V[(size_t)j * d + i];
                }
            } else if (!drop) {
                double w = (double)cnt[b] * exp(zb[b] - m);
                den += w;
                for (int i = 0; i < d; ++i) o[i] += w * vmean[(size_t)b * d + i];
            }
        }
        for (int i = 0; i < d; ++i) o[i] /= den;
        lse[g] = m + log(den);
    }
    free(zb);
    free(zt);
    free(sel);
}

/* ---- diagnostics (oracle only) ------------------------------------------------------------ */

/* Token-level distributions of one query head (Sec. 3.1, Eq. 1): P = softmax_j(z_j) and
 * Phat(S) = softmax_j(zhat_j), zhat_j = z_j in selected blocks and the block-mean logit
 * (arithmetic mean of the block's own logits) elsewhere.  Also the two normalisers of
 * App. A.1, returned as logs: logD = log sum_b Z_b, logDhat = log(sum_{b in S} Z_b + sum_{b not in S} |b| e^{zbar_b}).
 * drop != 0: Phat is the Drop distribution (zero outside S) and logDhat = log sum_{b in S} Z_b. */
void ckvo_token_dists(const float *qg, const float *K, int N, int d, int bs, const int *ids, int nsel,
                      double scale, int drop, double *P, double *Phat, double *logD, double *logDhat)
{
    int X = (N + bs - 1) / bs;
    char *sel = (char *)calloc((size_t)X, 1);
    for (int i = 0; i < nsel; ++i) sel[ids[i]] = 1;
    double *z = (double *)malloc(sizeof(double) * (size_t)N);
    double *zh = (double *)malloc(sizeof(double) * (size_t)N);
    double m = -INFINITY;
    for (int j = 0; j < N; ++j) {
        z[j] = dotf(qg, K + (size_t)j * d, d) * scale;
        if (z[j] > m) m = z[j];
    }
    for (int b = 0; b < X; ++b) {
        int lo = b * bs, hi = lo + bs < N ? lo + bs : N;
        double mean = 0.0;
        for (int j = lo; j < hi; ++j) mean += z[j];
        mean /= (hi - lo);
        for (int j = lo; j < hi; ++j) zh[j] = sel[b] ? z[j] : mean;
    }
    double D = 0.0, Dh = 0.0;
    for (int j = 0; j < N; ++j) {
        D += exp(z[j] - m);
        if (!drop || sel[j / bs]) Dh += exp(zh[j] - m);
    }
    for (int j = 0; j < N; ++j) {
        P[j] = exp(z[j] - m) / D;
        Phat[j] = (!drop || sel[j / bs]) ? exp(zh[j] - m) / Dh : 0.0;
    }
    *logD = m + log(D);
    *logDhat = m + log(Dh);
    free(zh);
    free(z);
    free(sel);
}

/* KL(A || B) = sum_j A_j log(A_j / B_j), by definition, with 0 log 0 = 0. */
double ckvo_kl(const double *A, const double *B, int n)
{
    double s = 0.0;
    for (int j = 0; j < n; ++j)
        if (A[j] > 0.0) s += A[j] * log(A[j] / B[j]);
    return s;
}

/* Exact per-block quantities of one query head (Eq. 3 and the exact residual of App. B.1):
 * p_b = Z_b / sum_c Z_c, sigma2_b = population variance of the block's logits,
 * rho_b = p_b (1 - |b| e^{zbar_b} / Z_b), ratio_b = Z_b / (|b| e^{zbar_b}), logZ_b = log Z_b. */
void ckvo_exact_blocks(const float *qg, const float *K, int N, int d, int bs, double scale,
                       double *p, double *sigma2, double *rho, double *ratio, double *logZ)
{
    int X = (N + bs - 1) / bs;
    double *z = (double *)malloc(sizeof(double) * (size_t)N);
    double m = -INFINITY;
    for (int j = 0; j < N; ++j) {
        z[j] = dotf(qg, K + (size_t)j * d, d) * scale;
        if (z[j] > m) m = z[j];
    }
    double D = 0.0;
    for (int j = 0; j < N; ++j) D += exp(z[j] - m);
    for (int b = 0; b < X; ++b) {
        int lo = b * bs, hi = lo + bs < N ? lo + bs : N;
        int n = hi - lo;
        double mean = 0.0, Zb = 0.0, var = 0.0;
        for (int j = lo; j < hi; ++j) mean += z[j];
        mean /= n;
        for (int j = lo; j < hi; ++j) {
            Zb += exp(z[j] - m);
            var += (z[j] - mean) * (z[j] - mean);
        }
        double meanw = (double)n * exp(mean - m);
        p[b] = Zb / D;
        sigma2[b] = var / n;
        rho[b] = p[b] * (1.0 - meanw / Zb);
        ratio[b] = Zb / meanw;
        logZ[b] = m + log(Zb);
    }
    free(z);
}
