/*
 * Reference oracle for Batch Normalization Sampling (arXiv 1810.10962).
 *
 * TEST INFRASTRUCTURE ONLY.  A plain, slow, double-precision CPU statement of what one BN layer
 * computes when its per-channel statistics come from a sampled subset of the activations.  It is
 * used by the tests, by the smoke check and by the benchmark's CPU-baseline leg; nothing in the
 * product path calls it and it shares no code with the CUDA library.
 *
 * Every function follows the paper's equations in the paper's order and notation:
 *   Eq. 1  normalise + affine          x^ = (x - E)/sqrt(Var + eps),  y = gamma x^ + beta
 *   Eq. 2  full statistics             E, Var over all m = N*H*W points of a feature map (1/m)
 *   Eq. 3  sampled statistics          E, Var over the s sampled points (1/s, biased)
 *   Eq. 5  BN backward                 dl/dx^, dl/dE, dl/dVar, dl/dx, dl/dgamma, dl/dbeta
 *   Eq. 6  BN-sampling backward        the dl/dE and dl/dVar terms reach x_i only if i is in S
 *   Algorithm 1  NS/BS slice  B[begin : begin+n_s-1, :, :, :]   (here: an explicit sample list)
 *   Algorithm 2  FS slice     B[:, bh : bh+h_s-1, bw : bw+w_s-1, :]
 *   Algorithm 3  VDN          statistics from the virtual rows only
 *   Eq. 4  VDN combined with a sampling rule   X = b X[x_v] + (1-b) X[x_s],  X in {E, Var}
 *   Eq. 8  moving average of E and Var for validation (Appendix D)
 * Layout is NCHW (the paper writes NHWC; the reduction is over N, H, W for each channel).
 *
 * Inputs are float arrays (bf16 data is widened exactly by the caller); all arithmetic is double.
 * No blocking, fusion or reordering: one channel at a time, loops in (n, h, w) order.
 * Channels are independent, so the channel loop may run on several host threads (OpenMP); that
 * changes no result.
 *
 * Parity pins (tests/test_oracle_*.py): sampling ratio 1 equals full BN and a library
 * batch-norm (forward and autograd backward); statistics equal numpy mean/var on the paper's
 * slices; the sampled set is standardised; central finite differences and an autograd pass through
 * an independently written forward confirm the backward; brute-force selection masks; the
 * m, s bookkeeping reproduces the one worked number the paper prints (Appendix C.1).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { RULE_FULL = 0, RULE_BATCH = 1, RULE_FEATURE = 2, RULE_VIRTUAL = 3 };
enum { OFFSETS_SHARED = 0, OFFSETS_PER_SAMPLE = 1, OFFSETS_PER_MAP = 2 };

typedef struct {
    int rule;
    int k;                      /* BATCH: number of sampled samples                     */
    const int32_t *sample_idx;  /* BATCH: k sample indices                              */
    int ph, pw;                 /* FEATURE: patch height and width                      */
    int offset_mode;            /* FEATURE: one (oh,ow) per layer / per sample / per map */
    const int32_t *offsets;     /* FEATURE: (oh,ow) pairs                               */
    int nv;                     /* VIRTUAL: number of virtual samples                   */
} oracle_sampling;

/* Is real element (n, c, h, w) a member of the sampled set S of its channel?  (VIRTUAL: S holds
 * only virtual elements, so no real element is a member.) */
static int in_S(const oracle_sampling *sp, int C, int n, int c, int h, int w)
{
    switch (sp->rule) {
    case RULE_FULL:
        return 1;
    case RULE_BATCH:
        for (int j = 0; j < sp->k; ++j)
            if (sp->sample_idx[j] == n) return 1;
        return 0;
    case RULE_FEATURE: {
        size_t e = 0;
        if (sp->offset_mode == OFFSETS_PER_SAMPLE) e = (size_t)n;
        if (sp->offset_mode == OFFSETS_PER_MAP) e = (size_t)n * C + c;
        int oh = sp->offsets[2 * e], ow = sp->offsets[2 * e + 1];
        return h >= oh && h < oh + sp->ph && w >= ow && w < ow + sp->pw;
    }
    default:
        return 0;
    }
}

/* s: the number of points that enter the statistics of one channel (Eq. 3). */
long long oracle_sample_count(int N, int H, int W, const oracle_sampling *sp)
{
    switch (sp->rule) {
    case RULE_FULL:    return (long long)N * H * W;
    case RULE_BATCH:   return (long long)sp->k * H * W;
    case RULE_FEATURE: return (long long)N * sp->ph * sp->pw;
    default:           return (long long)sp->nv * H * W;
    }
}

/* 1 where the element is sampled, 0 elsewhere; uint8 [N,C,H,W]. */
void oracle_selection_mask(int N, int C, int H, int W, const oracle_sampling *sp, uint8_t *mask)
{
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c)
            for (int h = 0; h < H; ++h)
                for (int w = 0; w < W; ++w)
                    mask[(((size_t)n * C + c) * H + h) * W + w] = (uint8_t)in_S(sp, C, n, c, h, w);
}

#define AT(n, c, h, w) ((((size_t)(n) * C + (c)) * H + (h)) * W + (w))
#define OUT(n, j, h, w) ((((size_t)(n) * nch + (j)) * H + (h)) * W + (w))

/*
 * Forward.  For each requested channel (channels[j], j < nch; NULL means all C channels in
 * order) computes E, Var (Eq. 3 over S; Eq. 2 when S is everything), invstd = 1/sqrt(Var + eps),
 * and y = gamma x^ + beta for every real element (Eq. 1); under VIRTUAL also yv for the virtual
 * rows when yv is not NULL.  Outputs are compact over the requested channels:
 * y [N,nch,H,W], yv [nv,nch,H,W], mean/var/invstd [nch].
 */
void oracle_forward(int N, int C, int H, int W, const float *x, const float *xv,
                    const float *gamma, const float *beta, double eps, const oracle_sampling *sp,
                    const int32_t *channels, int nch,
                    double *y, double *yv, double *mean, double *var, double *invstd)
{
    if (!channels) nch = C;
    const double s = (double)oracle_sample_count(N, H, W, sp);
#pragma omp parallel for schedule(dynamic, 1)
    for (int j = 0; j < nch; ++j) {
        const int c = channels ? channels[j] : j;
        /* Eq. 3, first half: E = (1/s) sum over S */
        double sum = 0.0;
        if (sp->rule == RULE_VIRTUAL) {
            for (int n = 0; n < sp->nv; ++n)
                for (int h = 0; h < H; ++h)
                    for (int w = 0; w < W; ++w) sum += (double)xv[AT(n, c, h, w)];
        } else {
            for (int n = 0; n < N; ++n)
                for (int h = 0; h < H; ++h)
                    for (int w = 0; w < W; ++w)
                        if (in_S(sp, C, n, c, h, w)) sum += (double)x[AT(n, c, h, w)];
        }
        const double E = sum / s;
        /* Eq. 3, second half: Var = (1/s) sum over S of (x - E)^2 */
        double sq = 0.0;
        if (sp->rule == RULE_VIRTUAL) {
            for (int n = 0; n < sp->nv; ++n)
                for (int h = 0; h < H; ++h)
                    for (int w = 0; w < W; ++w) {
                        double d = (double)xv[AT(n, c, h, w)] - E;
                        sq += d * d;
                    }
        } else {
            for (int n = 0; n < N; ++n)
                for (int h = 0; h < H; ++h)
                    for (int w = 0; w < W; ++w)
                        if (in_S(sp, C, n, c, h, w)) {
                            double d = (double)x[AT(n, c, h, w)] - E;
                            sq += d * d;
                        }
        }
        const double Var = sq / s;
        const double istd = 1.0 / sqrt(Var + eps);
        mean[j] = E;
        var[j] = Var;
        invstd[j] = istd;
        /* Eq. 1 for every element that is normalised with these statistics */
        const double g = (double)gamma[c], b = (double)beta[c];
        if (y)
            for (int n = 0; n < N; ++n)
                for (int h = 0; h < H; ++h)
                    for (int w = 0; w < W; ++w) {
                        double xhat = ((double)x[AT(n, c, h, w)] - E) * istd;
                        y[OUT(n, j, h, w)] = g * xhat + b;
                    }
        if (yv && sp->rule == RULE_VIRTUAL)
            for (int n = 0; n < sp->nv; ++n)
                for (int h = 0; h < H; ++h)
                    for (int w = 0; w < W; ++w) {
                        double xhat = ((double)xv[AT(n, c, h, w)] - E) * istd;
                        yv[OUT(n, j, h, w)] = g * xhat + b;
                    }
    }
}

/*
 * Backward (Eq. 5 and Eq. 6).  mean and var are the forward's statistics for the requested
 * channels ([nch], as oracle_forward returned them).  The sums of Eq. 5 run over every element
 * that was normalised with these statistics: all N*H*W real points and, under VIRTUAL with dyv
 * given, the virtual rows too (in the paper they are ordinary rows of the concatenated batch).
 * dx [N,nch,H,W]; dxv [nv,nch,H,W] (VIRTUAL, may be NULL); dgamma, dbeta [nch].
 */
void oracle_backward(int N, int C, int H, int W, const float *x, const float *xv,
                     const float *dy, const float *dyv, const float *gamma,
                     const double *mean, const double *var, double eps, const oracle_sampling *sp,
                     const int32_t *channels, int nch,
                     double *dx, double *dxv, double *dgamma, double *dbeta)
{
    if (!channels) nch = C;
    const double s = (double)oracle_sample_count(N, H, W, sp);
    const int virt = sp->rule == RULE_VIRTUAL;
#pragma omp parallel for schedule(dynamic, 1)
    for (int j = 0; j < nch; ++j) {
        const int c = channels ? channels[j] : j;
        const double E = mean[j], Var = var[j], g = (double)gamma[c];
        const double istd = 1.0 / sqrt(Var + eps);
        /* Eq. 5: the four sums keep their full length */
        double dl_dE = 0.0, dl_dVar = 0.0, dl_dgamma = 0.0, dl_dbeta = 0.0;
        for (int n = 0; n < N; ++n)
            for (int h = 0; h < H; ++h)
                for (int w = 0; w < W; ++w) {
                    double dyi = (double)dy[AT(n, c, h, w)], xi = (double)x[AT(n, c, h, w)];
                    double dl_dxhat = dyi * g;
                    dl_dE += dl_dxhat * (-1.0 / sqrt(Var + eps));
                    dl_dVar += dl_dxhat * (xi - E) * (-0.5) * pow(Var + eps, -1.5);
                    dl_dgamma += dyi * ((xi - E) * istd);
                    dl_dbeta += dyi;
                }
        if (virt && dyv)
            for (int n = 0; n < sp->nv; ++n)
                for (int h = 0; h < H; ++h)
                    for (int w = 0; w < W; ++w) {
                        double dyi = (double)dyv[AT(n, c, h, w)], xi = (double)xv[AT(n, c, h, w)];
                        double dl_dxhat = dyi * g;
                        dl_dE += dl_dxhat * (-1.0 / sqrt(Var + eps));
                        dl_dVar += dl_dxhat * (xi - E) * (-0.5) * pow(Var + eps, -1.5);
                        dl_dgamma += dyi * ((xi - E) * istd);
                        dl_dbeta += dyi;
                    }
        dgamma[j] = dl_dgamma;
        dbeta[j] = dl_dbeta;
        /* Eq. 6: upper branch on S, lower branch elsewhere */
        if (dx)
            for (int n = 0; n < N; ++n)
                for (int h = 0; h < H; ++h)
                    for (int w = 0; w < W; ++w) {
                        double dyi = (double)dy[AT(n, c, h, w)], xi = (double)x[AT(n, c, h, w)];
                        double dl_dxhat = dyi * g;
                        double v = dl_dxhat / sqrt(Var + eps);
                        if (in_S(sp, C, n, c, h, w))
                            v += dl_dE * (1.0 / s) + dl_dVar * (2.0 * (xi - E) / s);
                        dx[OUT(n, j, h, w)] = v;
                    }
        /* the virtual rows are all members of S */
        if (virt && dxv)
            for (int n = 0; n < sp->nv; ++n)
                for (int h = 0; h < H; ++h)
                    for (int w = 0; w < W; ++w) {
                        double dyi = dyv ? (double)dyv[AT(n, c, h, w)] : 0.0;
                        double xi = (double)xv[AT(n, c, h, w)];
                        double dl_dxhat = dyi * g;
                        dxv[OUT(n, j, h, w)] = dl_dxhat / sqrt(Var + eps) + dl_dE * (1.0 / s) +
                                               dl_dVar * (2.0 * (xi - E) / s);
                    }
    }
}

/* Host threads the channel loops run on (1 without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
int oracle_threads(void) { return omp_get_max_threads(); }
#else
int oracle_threads(void) { return 1; }
#endif

/* Appendix C.1: with an adder tree the depth falls from log(m) to log(s), a ratio of log_s(m). */
double oracle_adder_tree_depth_ratio(int N, int H, int W, const oracle_sampling *sp)
{
    double m = (double)N * H * W;
    double s = (double)oracle_sample_count(N, H, W, sp);
    return log(m) / log(s);
}

/* ------------------------------------------------------------------------------------------------
 * Eq. 4: statistics mixed from the virtual samples and a sampling rule of the real batch,
 *   E = b E[x_v] + (1-b) E[x_s],   Var = b Var[x_v] + (1-b) Var[x_s]
 * where each variance is taken about its own mean (Eq. 3 applied to each set).  sp is the rule of
 * the real batch (BATCH or FEATURE); the virtual set is all of xv [nv,C,H,W].  Every real and every
 * virtual element is normalised with the mixed statistics (Eq. 1).
 * Outputs, compact over the requested channels: y [N,nch,H,W], yv [nv,nch,H,W] (may be NULL),
 * mean/var (mixed), mean_s/var_s (sampled real set), mean_v/var_v (virtual set), each [nch].
 */
void oracle_forward_mixed(int N, int C, int H, int W, const float *x, const float *xv, int nv,
                          const float *gamma, const float *beta, double eps, double b,
                          const oracle_sampling *sp, const int32_t *channels, int nch,
                          double *y, double *yv, double *mean, double *var,
                          double *mean_s, double *var_s, double *mean_v, double *var_v)
{
    if (!channels) nch = C;
    const double s_s = (double)oracle_sample_count(N, H, W, sp);
    const double s_v = (double)nv * H * W;
#pragma omp parallel for schedule(dynamic, 1)
    for (int j = 0; j < nch; ++j) {
        const int c = channels ? channels[j] : j;
        /* Eq. 3 on the sampled real set */
        double sum = 0.0, sq = 0.0;
        for (int n = 0; n < N; ++n)
            for (int h = 0; h < H; ++h)
                for (int w = 0; w < W; ++w)
                    if (in_S(sp, C, n, c, h, w)) sum += (double)x[AT(n, c, h, w)];
        const double E_s = sum / s_s;
        for (int n = 0; n < N; ++n)
            for (int h = 0; h < H; ++h)
                for (int w = 0; w < W; ++w)
                    if (in_S(sp, C, n, c, h, w)) {
                        double d = (double)x[AT(n, c, h, w)] - E_s;
                        sq += d * d;
                    }
        const double Var_s = sq / s_s;
        /* Eq. 3 on the virtual set */
        sum = 0.0, sq = 0.0;
        for (int n = 0; n < nv; ++n)
            for (int h = 0; h < H; ++h)
                for (int w = 0; w < W; ++w) sum += (double)xv[AT(n, c, h, w)];
        const double E_v = sum / s_v;
        for (int n = 0; n < nv; ++n)
            for (int h = 0; h < H; ++h)
                for (int w = 0; w < W; ++w) {
                    double d = (double)xv[AT(n, c, h, w)] - E_v;
                    sq += d * d;
                }
        const double Var_v = sq / s_v;
        /* Eq. 4 */
        const double E = b * E_v + (1.0 - b) * E_s;
        const double Var = b * Var_v + (1.0 - b) * Var_s;
        mean[j] = E, var[j] = Var;
        mean_s[j] = E_s, var_s[j] = Var_s;
        mean_v[j] = E_v, var_v[j] = Var_v;
        /* Eq. 1 */
        const double g = (double)gamma[c], bt = (double)beta[c];
        if (y)
            for (int n = 0; n < N; ++n)
                for (int h = 0; h < H; ++h)
                    for (int w = 0; w < W; ++w)
                        y[OUT(n, j, h, w)] = g * (((double)x[AT(n, c, h, w)] - E) / sqrt(Var + eps)) + bt;
        if (yv)
            for (int n = 0; n < nv; ++n)
                for (int h = 0; h < H; ++h)
                    for (int w = 0; w < W; ++w)
                        yv[OUT(n, j, h, w)] = g * (((double)xv[AT(n, c, h, w)] - E) / sqrt(Var + eps)) + bt;
    }
}

/*
 * Backward of the mixed statistics, by the chain rule through Eq. 4 in the notation of Eq. 5/6.
 * dl/dE and dl/dVar are the full-length sums of Eq. 5 over every normalised element (the real batch
 * and, when dyv is given, the virtual rows).  Var does not depend on E here (each variance is about
 * its own mean), and d Var_s / d E_s = -(2/s_s) sum_S (x - E_s) = 0, so
 *   dl/dE_s = (1-b) dl/dE,  dl/dVar_s = (1-b) dl/dVar,  dl/dE_v = b dl/dE,  dl/dVar_v = b dl/dVar,
 *   dx_i  = dl/dx^_i / sqrt(Var+eps) + [i in S] ( dl/dE_s / s_s + dl/dVar_s 2 (x_i - E_s) / s_s )
 *   dxv_i = dl/dx^v_i / sqrt(Var+eps) +           dl/dE_v / s_v + dl/dVar_v 2 (xv_i - E_v) / s_v
 */
void oracle_backward_mixed(int N, int C, int H, int W, const float *x, const float *xv, int nv,
                           const float *dy, const float *dyv, const float *gamma,
                           const double *mean, const double *var, const double *mean_s, const double *mean_v,
                           double eps, double b, const oracle_sampling *sp,
                           const int32_t *channels, int nch,
                           double *dx, double *dxv, double *dgamma, double *dbeta)
{
    if (!channels) nch = C;
    const double s_s = (double)oracle_sample_count(N, H, W, sp);
    const double s_v = (double)nv * H * W;
#pragma omp parallel for schedule(dynamic, 1)
    for (int j = 0; j < nch; ++j) {
        const int c = channels ? channels[j] : j;
        const double E = mean[j], Var = var[j], E_s = mean_s[j], E_v = mean_v[j], g = (double)gamma[c];
        double dl_dE = 0.0, dl_dVar = 0.0, dl_dgamma = 0.0, dl_dbeta = 0.0;
        for (int n = 0; n < N; ++n)
            for (int h = 0; h < H; ++h)
                for (int w = 0; w < W; ++w) {
                    double dyi = (double)dy[AT(n, c, h, w)], xi = (double)x[AT(n, c, h, w)];
                    double dl_dxhat = dyi * g;
                    dl_dE += dl_dxhat * (-1.0 / sqrt(Var + eps));
                    dl_dVar += dl_dxhat * (xi - E) * (-0.5) * pow(Var + eps, -1.5);
                    dl_dgamma += dyi * ((xi - E) / sqrt(Var + eps));
                    dl_dbeta += dyi;
                }
        if (dyv)
            for (int n = 0; n < nv; ++n)
                for (int h = 0; h < H; ++h)
                    for (int w = 0; w < W; ++w) {
                        double dyi = (double)dyv[AT(n, c, h, w)], xi = (double)xv[AT(n, c, h, w)];
                        double dl_dxhat = dyi * g;
                        dl_dE += dl_dxhat * (-1.0 / sqrt(Var + eps));
                        dl_dVar += dl_dxhat * (xi - E) * (-0.5) * pow(Var + eps, -1.5);
                        dl_dgamma += dyi * ((xi - E) / sqrt(Var + eps));
                        dl_dbeta += dyi;
                    }
        dgamma[j] = dl_dgamma;
        dbeta[j] = dl_dbeta;
        const double dl_dE_s = (1.0 - b) * dl_dE, dl_dVar_s = (1.0 - b) * dl_dVar;
        const double dl_dE_v = b * dl_dE, dl_dVar_v = b * dl_dVar;
        if (dx)
            for (int n = 0; n < N; ++n)
                for (int h = 0; h < H; ++h)
                    for (int w = 0; w < W; ++w) {
                        double dyi = (double)dy[AT(n, c, h, w)], xi = (double)x[AT(n, c, h, w)];
                        double v = dyi * g / sqrt(Var + eps);
                        if (in_S(sp, C, n, c, h, w)) v += dl_dE_s / s_s + dl_dVar_s * 2.0 * (xi - E_s) / s_s;
                        dx[OUT(n, j, h, w)] = v;
                    }
        if (dxv)
            for (int n = 0; n < nv; ++n)
                for (int h = 0; h < H; ++h)
                    for (int w = 0; w < W; ++w) {
                        double dyi = dyv ? (double)dyv[AT(n, c, h, w)] : 0.0;
                        double xi = (double)xv[AT(n, c, h, w)];
                        dxv[OUT(n, j, h, w)] = dyi * g / sqrt(Var + eps) + dl_dE_v / s_v +
                                               dl_dVar_v * 2.0 * (xi - E_v) / s_v;
                    }
    }
}

/* ------------------------------------------------------------------------------------------------
 * Appendix D, Eq. 8: the recorded moving average of a statistic X (E or Var) over iterations:
 * X_ma = X at the first iteration, alpha X + (1 - alpha) X_ma afterwards (alpha weights the NEW value).
 */
void oracle_moving_average(int C, int first_iteration, double alpha, const double *X, double *X_ma)
{
    for (int c = 0; c < C; ++c) X_ma[c] = first_iteration ? X[c] : alpha * X[c] + (1.0 - alpha) * X_ma[c];
}

/* Validation step (Appendix D): Eq. 1 with E and Var replaced by the recorded moving averages. */
void oracle_inference_forward(int N, int C, int H, int W, const float *x, const float *gamma,
                              const float *beta, double eps, const double *E_ma, const double *Var_ma,
                              double *y)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int c = 0; c < C; ++c)
        for (int n = 0; n < N; ++n)
            for (int h = 0; h < H; ++h)
                for (int w = 0; w < W; ++w) {
                    double xhat = ((double)x[AT(n, c, h, w)] - E_ma[c]) / sqrt(Var_ma[c] + eps);
                    y[AT(n, c, h, w)] = (double)gamma[c] * xhat + (double)beta[c];
                }
}
