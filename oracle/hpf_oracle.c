/*
 * hpf_oracle.c -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, fp64 CPU statement of what the partitioned, micro-batch
 * pipelined training step of HyPar-Flow (arXiv 1911.05146) computes for a
 * convolutional network given as a list of ops.  It exists so that the CUDA
 * library can be checked element by element.  Only tests, the smoke entry and
 * the benchmark's CPU-baseline leg may call it.  It shares no code with the
 * CUDA library and includes none of its headers.
 *
 * What the paper fixes, and where:
 *   - Section 5.1: the model is a list of layers; every process owns a
 *     consecutive group of them (a "model partition") plus the lists that say
 *     which layer feeds which.
 *   - Section 5.2, Eq. 1-7: back-propagation across a partition boundary.  The
 *     partition that owns the later layers computes its own weight gradients
 *     (Eq. 5) and the "partial error" dL/d(boundary activation) (Eq. 7); the
 *     earlier partition finishes the chain rule with it (Eq. 6).
 *   - Section 5.3: forward send/recv of "partial predictions" (activations),
 *     backward send/recv of partial errors, skip connections that cross a
 *     boundary (Forward/Backward lists), gradients accumulated (averaged),
 *     and the batch split into pipeline stages (micro-batches).
 * The method reaches exactly the result of ordinary back-propagation applied
 * to each micro-batch, so this file is that definition written out: a forward
 * sweep in list order, a reverse sweep, one gradient slot per micro-batch, and
 * the average.  A second routine executes the same sweep partition by
 * partition through explicit mailboxes (the send/recv of Section 5.3) and must
 * give bit-identical numbers.
 *
 * Readings taken where the paper is silent (listed in the design notes):
 * batch-norm statistics are per micro-batch with the biased variance; the loss
 * is softmax cross-entropy, mean over the micro-batch; the step's gradient is
 * (1/M) * sum over micro-batches in ascending order; ReLU derivative at 0 is
 * 0; convolutions are cross-correlations with zero padding and no bias; a
 * tensor with several consumers sums their gradients in descending consumer
 * order; max-pool padding is -infinity and ties go to the first window
 * position in row-major order.
 *
 * ReLU decisions.  The derivative of ReLU is a step, so dL/d(anything upstream)
 * is a discontinuous function of the forward values: an implementation whose
 * pre-activation z differs from this file's by a rounding error takes the
 * other branch wherever |z| is smaller than that error, and both branches are
 * correct results of the method in their own arithmetic.  The sweeps therefore
 * accept, per BNRELU op, the decisions (z > 0) another implementation took:
 * where |z| >= tau*|gamma_c| the decision is unique and this file's own is
 * used (a disagreement there is counted as a violation); where |z| is below
 * that window the supplied decision is used.  With no decisions supplied, or
 * tau = 0, nothing changes.
 *
 * Layout: activations are [n][h][w][c] (channels innermost), convolution
 * weights [c_out][r][s][c_in].  Everything is double.
 *
 * Pinned by tests/test_oracle_*.py (finite differences, adjoint identities,
 * closed forms, partition and micro-batch invariance, a library cross-check).
 * The paper prints no activation, loss or gradient value, so agreement with
 * the authors' own runs is "parity unpinned" and cannot be otherwise.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* BN = batch normalisation without the activation, RELU = the activation alone: the post-activation (v1) residual
 * block is conv-BN-RELU-conv-BN, ADD with the shortcut, RELU. */
enum { ORA_CONV = 1, ORA_BNRELU = 2, ORA_ADD = 3, ORA_MAXPOOL = 4, ORA_HEAD = 5, ORA_BN = 6, ORA_RELU = 7 };
enum { ORA_OK = 0, ORA_EINVAL = -1, ORA_ENOMEM = -2 };

typedef struct {
    int32_t kind;        /* ORA_* */
    int32_t src0, src1;  /* producing op, -1 = network input; src1 only for ADD */
    int32_t c_in, c_out; /* HEAD: c_out = number of classes */
    int32_t ksize, stride, pad;
    double eps;          /* BNRELU */
} ora_op;

/* ------------------------------------------------------------------ */
/* Integer bookkeeping (Section 5.1: local layers and dependency lists) */
/* ------------------------------------------------------------------ */

/* Output (H, W, C) of every op.  Also validates the list. */
int ora_shapes(const ora_op *ops, int32_t n_ops, const int32_t in_hwc[3], int32_t *out_hwc)
{
    if (!ops || !in_hwc || !out_hwc || n_ops < 1) return ORA_EINVAL;
    for (int32_t i = 0; i < n_ops; ++i) {
        const ora_op *o = &ops[i];
        if (o->src0 < -1 || o->src0 >= i) return ORA_EINVAL;
        const int32_t *s = o->src0 < 0 ? in_hwc : &out_hwc[3 * o->src0];
        if (o->src0 >= 0 && ops[o->src0].kind == ORA_HEAD) return ORA_EINVAL;
        int32_t H = s[0], W = s[1], C = s[2];
        int32_t *d = &out_hwc[3 * i];
        switch (o->kind) {
        case ORA_CONV:
        case ORA_MAXPOOL:
            if (o->c_in != C || o->ksize < 1 || o->stride < 1 || o->pad < 0) return ORA_EINVAL;
            if (o->kind == ORA_MAXPOOL && o->c_out != C) return ORA_EINVAL;
            if (o->c_out < 1 || H + 2 * o->pad < o->ksize || W + 2 * o->pad < o->ksize) return ORA_EINVAL;
            d[0] = (H + 2 * o->pad - o->ksize) / o->stride + 1;
            d[1] = (W + 2 * o->pad - o->ksize) / o->stride + 1;
            d[2] = o->c_out;
            break;
        case ORA_BNRELU:
        case ORA_BN:
        case ORA_RELU:
            if (o->c_in != C || o->c_out != C) return ORA_EINVAL;
            d[0] = H; d[1] = W; d[2] = C;
            break;
        case ORA_ADD: {
            if (o->src1 < -1 || o->src1 >= i) return ORA_EINVAL;
            const int32_t *t = o->src1 < 0 ? in_hwc : &out_hwc[3 * o->src1];
            if (t[0] != H || t[1] != W || t[2] != C || o->c_out != C) return ORA_EINVAL;
            d[0] = H; d[1] = W; d[2] = C;
            break;
        }
        case ORA_HEAD:
            if (i != n_ops - 1 || o->c_in != C || o->c_out < 1) return ORA_EINVAL;
            d[0] = 1; d[1] = 1; d[2] = o->c_out;
            break;
        default:
            return ORA_EINVAL;
        }
    }
    if (ops[n_ops - 1].kind != ORA_HEAD) return ORA_EINVAL;
    return ORA_OK;
}

/* Offsets into the flat parameter vector: ops in list order; CONV weights
 * [c_out][r][s][c_in]; BNRELU gamma then beta; HEAD W[classes][C] then bias. */
int ora_param_layout(const ora_op *ops, int32_t n_ops, int64_t *w_off, int64_t *w_cnt,
                     int64_t *b_off, int64_t *b_cnt, int64_t *total)
{
    int64_t at = 0;
    for (int32_t i = 0; i < n_ops; ++i) {
        const ora_op *o = &ops[i];
        int64_t wc = 0, bc = 0;
        if (o->kind == ORA_CONV) wc = (int64_t)o->c_out * o->ksize * o->ksize * o->c_in;
        else if (o->kind == ORA_BNRELU || o->kind == ORA_BN) { wc = o->c_in; bc = o->c_in; }
        else if (o->kind == ORA_HEAD) { wc = (int64_t)o->c_out * o->c_in; bc = o->c_out; }
        w_off[i] = at; w_cnt[i] = wc; at += wc;
        b_off[i] = at; b_cnt[i] = bc; at += bc;
    }
    *total = at;
    return ORA_OK;
}

/* cuts: P-1 strictly increasing op indices in [1, n_ops-1]; partition p owns
 * ops [cut[p-1], cut[p]) with cut[-1] = 0 and cut[P-1] = n_ops. */
int ora_check_cuts(int32_t n_ops, const int32_t *cuts, int32_t n_cuts)
{
    if (n_cuts < 0 || n_cuts > n_ops - 1) return ORA_EINVAL;
    for (int32_t j = 0; j < n_cuts; ++j) {
        if (cuts[j] < 1 || cuts[j] > n_ops - 1) return ORA_EINVAL;
        if (j && cuts[j] <= cuts[j - 1]) return ORA_EINVAL;
    }
    return ORA_OK;
}

int ora_partition_of_ops(int32_t n_ops, const int32_t *cuts, int32_t n_cuts, int32_t *part_of_op)
{
    if (ora_check_cuts(n_ops, cuts, n_cuts)) return ORA_EINVAL;
    int32_t p = 0;
    for (int32_t i = 0; i < n_ops; ++i) {
        while (p < n_cuts && i >= cuts[p]) ++p;
        part_of_op[i] = p;
    }
    return ORA_OK;
}

/* The tensors that cross a cut placed before op `cut`: produced by an op
 * before the cut and read by an op at or after it (the trunk and, when the cut
 * falls inside a residual block, the shortcut).  Ascending producer index. */
int ora_live_set(const ora_op *ops, int32_t n_ops, int32_t cut, int32_t *producers, int32_t *count)
{
    int32_t n = 0;
    for (int32_t t = 0; t < cut; ++t) {
        int live = 0;
        for (int32_t i = cut; i < n_ops && !live; ++i) {
            if (ops[i].src0 == t) live = 1;
            if (ops[i].kind == ORA_ADD && ops[i].src1 == t) live = 1;
        }
        if (live) producers[n++] = t;
    }
    *count = n;
    return ORA_OK;
}

/* Micro-batch m is the samples [m*b, (m+1)*b), b = B/M (Section 5.3, pipelining). */
int ora_microbatch_range(int32_t B, int32_t M, int32_t m, int32_t *first, int32_t *end)
{
    if (M < 1 || B < 1 || B % M || m < 0 || m >= M) return ORA_EINVAL;
    int32_t b = B / M;
    *first = m * b; *end = (m + 1) * b;
    return ORA_OK;
}

/* Fill/drain pipeline: forward (p,m) at tick p+m, backward (p,m) at tick
 * (P-1-p)+m counted from the start of the backward phase. */
int ora_schedule_tick(int32_t P, int32_t M, int32_t p, int32_t m, int32_t *fwd, int32_t *bwd)
{
    if (p < 0 || p >= P || m < 0 || m >= M) return ORA_EINVAL;
    *fwd = p + m; *bwd = (P - 1 - p) + m;
    return ORA_OK;
}

/* ------------------------------------------------------------------ */
/* Ops, forward and backward                                           */
/* ------------------------------------------------------------------ */

/* y[n,p,q,k] = sum_{r,s,c} x[n, p*st+r-pad, q*st+s-pad, c] * w[k,r,s,c] */
void ora_conv_fwd(const double *x, int32_t N, int32_t H, int32_t W, int32_t C,
                  const double *w, int32_t K, int32_t R, int32_t st, int32_t pad, double *y)
{
    int32_t P = (H + 2 * pad - R) / st + 1, Q = (W + 2 * pad - R) / st + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int32_t n = 0; n < N; ++n)
        for (int32_t p = 0; p < P; ++p)
            for (int32_t q = 0; q < Q; ++q)
                for (int32_t k = 0; k < K; ++k) {
                    double acc = 0.0;
                    for (int32_t r = 0; r < R; ++r) {
                        int32_t ih = p * st + r - pad;
                        if (ih < 0 || ih >= H) continue;
                        for (int32_t s = 0; s < R; ++s) {
                            int32_t iw = q * st + s - pad;
                            if (iw < 0 || iw >= W) continue;
                            const double *xr = &x[(((int64_t)n * H + ih) * W + iw) * C];
                            const double *wr = &w[(((int64_t)k * R + r) * R + s) * C];
                            for (int32_t c = 0; c < C; ++c) acc += xr[c] * wr[c];
                        }
                    }
                    y[(((int64_t)n * P + p) * Q + q) * K + k] = acc;
                }
}

/* dx[n,h,w,c] = sum over (k,r,s) and the (p,q) with h = p*st+r-pad, w = q*st+s-pad
 * of dy[n,p,q,k] * w[k,r,s,c].  Overwrites dx. */
void ora_conv_dgrad(const double *dy, int32_t N, int32_t H, int32_t W, int32_t C,
                    const double *w, int32_t K, int32_t R, int32_t st, int32_t pad, double *dx)
{
    int32_t P = (H + 2 * pad - R) / st + 1, Q = (W + 2 * pad - R) / st + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int32_t n = 0; n < N; ++n)
        for (int32_t h = 0; h < H; ++h)
            for (int32_t ww = 0; ww < W; ++ww) {
                double *dxr = &dx[(((int64_t)n * H + h) * W + ww) * C];
                for (int32_t c = 0; c < C; ++c) dxr[c] = 0.0;
                for (int32_t r = 0; r < R; ++r) {
                    int32_t tp = h + pad - r;
                    if (tp < 0 || tp % st) continue;
                    int32_t p = tp / st;
                    if (p >= P) continue;
                    for (int32_t s = 0; s < R; ++s) {
                        int32_t tq = ww + pad - s;
                        if (tq < 0 || tq % st) continue;
                        int32_t q = tq / st;
                        if (q >= Q) continue;
                        const double *dyr = &dy[(((int64_t)n * P + p) * Q + q) * K];
                        for (int32_t k = 0; k < K; ++k) {
                            double d = dyr[k];
                            const double *wr = &w[(((int64_t)k * R + r) * R + s) * C];
                            for (int32_t c = 0; c < C; ++c) dxr[c] += d * wr[c];
                        }
                    }
                }
            }
}

/* dw[k,r,s,c] = sum_{n,p,q} dy[n,p,q,k] * x[n, p*st+r-pad, q*st+s-pad, c].  Overwrites dw. */
void ora_conv_wgrad(const double *x, int32_t N, int32_t H, int32_t W, int32_t C,
                    const double *dy, int32_t K, int32_t R, int32_t st, int32_t pad, double *dw)
{
    int32_t P = (H + 2 * pad - R) / st + 1, Q = (W + 2 * pad - R) / st + 1;
#pragma omp parallel for schedule(static)
    for (int32_t k = 0; k < K; ++k) {
        double *dwk = &dw[(int64_t)k * R * R * C];
        for (int64_t j = 0; j < (int64_t)R * R * C; ++j) dwk[j] = 0.0;
        for (int32_t n = 0; n < N; ++n)
            for (int32_t p = 0; p < P; ++p)
                for (int32_t q = 0; q < Q; ++q) {
                    double d = dy[(((int64_t)n * P + p) * Q + q) * K + k];
                    for (int32_t r = 0; r < R; ++r) {
                        int32_t ih = p * st + r - pad;
                        if (ih < 0 || ih >= H) continue;
                        for (int32_t s = 0; s < R; ++s) {
                            int32_t iw = q * st + s - pad;
                            if (iw < 0 || iw >= W) continue;
                            const double *xr = &x[(((int64_t)n * H + ih) * W + iw) * C];
                            double *dwr = &dwk[((int64_t)r * R + s) * C];
                            for (int32_t c = 0; c < C; ++c) dwr[c] += d * xr[c];
                        }
                    }
                }
    }
}

/* Per-channel mean and biased variance over `rows` = n*h*w positions. */
void ora_bn_stats(const double *x, int64_t rows, int32_t C, double *mean, double *var)
{
#pragma omp parallel for schedule(static)
    for (int32_t c = 0; c < C; ++c) {
        double s = 0.0;
        for (int64_t i = 0; i < rows; ++i) s += x[i * C + c];
        double mu = s / (double)rows, v = 0.0;
        for (int64_t i = 0; i < rows; ++i) { double d = x[i * C + c] - mu; v += d * d; }
        mean[c] = mu; var[c] = v / (double)rows;
    }
}

/* y = max(0, gamma * (x - mean) / sqrt(var + eps) + beta) */
void ora_bnrelu_fwd(const double *x, int64_t rows, int32_t C, const double *gamma, const double *beta,
                    double eps, double *y)
{
    double *mean = (double *)malloc(sizeof(double) * 2 * (size_t)C), *var = mean + C;
    ora_bn_stats(x, rows, C, mean, var);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < rows; ++i)
        for (int32_t c = 0; c < C; ++c) {
            double xh = (x[i * C + c] - mean[c]) / sqrt(var[c] + eps);
            double z = gamma[c] * xh + beta[c];
            y[i * C + c] = z > 0.0 ? z : 0.0;
        }
    free(mean);
}

/* dz = dy * [gamma*xhat+beta > 0]; dbeta = sum dz; dgamma = sum dz*xhat;
 * dx = gamma / sqrt(var+eps) * (dz - dbeta/rows - xhat * dgamma/rows).
 * decisions (may be NULL): one byte per element, nonzero = "z > 0" as another
 * implementation decided it; honoured only inside the window |z| < tau*|gamma_c|.
 * counts (may be NULL): [0] += decisions used that differ from this file's own,
 * [1] += supplied decisions that differ outside the window (violations). */
void ora_bnrelu_bwd_dec(const double *x, const double *dy, int64_t rows, int32_t C, const double *gamma,
                        const double *beta, double eps, const uint8_t *decisions, double tau, int64_t *counts,
                        double *dx, double *dgamma, double *dbeta)
{
    double *mean = (double *)malloc(sizeof(double) * 2 * (size_t)C), *var = mean + C;
    int64_t n_used = 0, n_viol = 0;
    ora_bn_stats(x, rows, C, mean, var);
#pragma omp parallel for schedule(static) reduction(+ : n_used, n_viol)
    for (int32_t c = 0; c < C; ++c) {
        double rstd = 1.0 / sqrt(var[c] + eps), sb = 0.0, sg = 0.0;
        double window = tau * fabs(gamma[c]);
        uint8_t *open = (uint8_t *)malloc((size_t)rows);
        for (int64_t i = 0; i < rows; ++i) {
            double xh = (x[i * C + c] - mean[c]) * rstd;
            double z = gamma[c] * xh + beta[c];
            int own = z > 0.0;
            int use = own;
            if (decisions) {
                int theirs = decisions[i * C + c] != 0;
                if (theirs != own) {
                    if (fabs(z) < window) { use = theirs; ++n_used; }
                    else ++n_viol;
                }
            }
            open[i] = (uint8_t)use;
            double dz = use ? dy[i * C + c] : 0.0;
            sb += dz; sg += dz * xh;
        }
        dbeta[c] = sb; dgamma[c] = sg;
        for (int64_t i = 0; i < rows; ++i) {
            double xh = (x[i * C + c] - mean[c]) * rstd;
            double dz = open[i] ? dy[i * C + c] : 0.0;
            dx[i * C + c] = gamma[c] * rstd * (dz - sb / (double)rows - xh * sg / (double)rows);
        }
        free(open);
    }
    if (counts) { counts[0] += n_used; counts[1] += n_viol; }
    free(mean);
}

void ora_bnrelu_bwd(const double *x, const double *dy, int64_t rows, int32_t C, const double *gamma,
                    const double *beta, double eps, double *dx, double *dgamma, double *dbeta)
{
    ora_bnrelu_bwd_dec(x, dy, rows, C, gamma, beta, eps, NULL, 0.0, NULL, dx, dgamma, dbeta);
}

/* Batch normalisation alone: y = gamma * (x - mean) / sqrt(var + eps) + beta (per-micro-batch statistics, biased
 * variance), and its backward dx = gamma / sqrt(var+eps) * (dy - mean(dy) - xhat * mean(dy*xhat)). */
void ora_bn_fwd(const double *x, int64_t rows, int32_t C, const double *gamma, const double *beta, double eps, double *y)
{
    double *mean = (double *)malloc(sizeof(double) * 2 * (size_t)C), *var = mean + C;
    ora_bn_stats(x, rows, C, mean, var);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < rows; ++i)
        for (int32_t c = 0; c < C; ++c)
            y[i * C + c] = gamma[c] * ((x[i * C + c] - mean[c]) / sqrt(var[c] + eps)) + beta[c];
    free(mean);
}

void ora_bn_bwd(const double *x, const double *dy, int64_t rows, int32_t C, const double *gamma, double eps,
                double *dx, double *dgamma, double *dbeta)
{
    double *mean = (double *)malloc(sizeof(double) * 2 * (size_t)C), *var = mean + C;
    ora_bn_stats(x, rows, C, mean, var);
#pragma omp parallel for schedule(static)
    for (int32_t c = 0; c < C; ++c) {
        double rstd = 1.0 / sqrt(var[c] + eps), sb = 0.0, sg = 0.0;
        for (int64_t i = 0; i < rows; ++i) {
            double xh = (x[i * C + c] - mean[c]) * rstd;
            sb += dy[i * C + c]; sg += dy[i * C + c] * xh;
        }
        dbeta[c] = sb; dgamma[c] = sg;
        for (int64_t i = 0; i < rows; ++i) {
            double xh = (x[i * C + c] - mean[c]) * rstd;
            dx[i * C + c] = gamma[c] * rstd * (dy[i * C + c] - sb / (double)rows - xh * sg / (double)rows);
        }
    }
    free(mean);
}

/* y = max(x, 0) and dx = dy * [x > 0] (derivative 0 at 0).  decisions / tau / counts as in ora_bnrelu_bwd_dec,
 * the window being |x| < tau. */
void ora_relu_fwd(const double *x, int64_t n, double *y)
{
    for (int64_t i = 0; i < n; ++i) y[i] = x[i] > 0.0 ? x[i] : 0.0;
}

void ora_relu_bwd_dec(const double *x, const double *dy, int64_t n, const uint8_t *decisions, double tau,
                      int64_t *counts, double *dx)
{
    int64_t n_used = 0, n_viol = 0;
    for (int64_t i = 0; i < n; ++i) {
        int own = x[i] > 0.0, use = own;
        if (decisions) {
            int theirs = decisions[i] != 0;
            if (theirs != own) {
                if (fabs(x[i]) < tau) { use = theirs; ++n_used; }
                else ++n_viol;
            }
        }
        dx[i] = use ? dy[i] : 0.0;
    }
    if (counts) { counts[0] += n_used; counts[1] += n_viol; }
}

/* Window max with -infinity padding; argmax = first maximum in (r,s) row-major order. */
void ora_maxpool_fwd(const double *x, int32_t N, int32_t H, int32_t W, int32_t C, int32_t R, int32_t st,
                     int32_t pad, double *y)
{
    int32_t P = (H + 2 * pad - R) / st + 1, Q = (W + 2 * pad - R) / st + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int32_t n = 0; n < N; ++n)
        for (int32_t p = 0; p < P; ++p)
            for (int32_t q = 0; q < Q; ++q)
                for (int32_t c = 0; c < C; ++c) {
                    double best = -INFINITY;
                    for (int32_t r = 0; r < R; ++r) {
                        int32_t ih = p * st + r - pad;
                        if (ih < 0 || ih >= H) continue;
                        for (int32_t s = 0; s < R; ++s) {
                            int32_t iw = q * st + s - pad;
                            if (iw < 0 || iw >= W) continue;
                            double v = x[(((int64_t)n * H + ih) * W + iw) * C + c];
                            if (v > best) best = v;
                        }
                    }
                    y[(((int64_t)n * P + p) * Q + q) * C + c] = best;
                }
}

/* dx[argmax window position] += dy; overwrites dx (zero elsewhere). */
void ora_maxpool_bwd(const double *x, const double *dy, int32_t N, int32_t H, int32_t W, int32_t C,
                     int32_t R, int32_t st, int32_t pad, double *dx)
{
    int32_t P = (H + 2 * pad - R) / st + 1, Q = (W + 2 * pad - R) / st + 1;
    memset(dx, 0, sizeof(double) * (size_t)N * H * W * C);
#pragma omp parallel for schedule(static)
    for (int32_t n = 0; n < N; ++n)
        for (int32_t p = 0; p < P; ++p)
            for (int32_t q = 0; q < Q; ++q)
                for (int32_t c = 0; c < C; ++c) {
                    double best = -INFINITY;
                    int64_t at = -1;
                    for (int32_t r = 0; r < R; ++r) {
                        int32_t ih = p * st + r - pad;
                        if (ih < 0 || ih >= H) continue;
                        for (int32_t s = 0; s < R; ++s) {
                            int32_t iw = q * st + s - pad;
                            if (iw < 0 || iw >= W) continue;
                            int64_t j = (((int64_t)n * H + ih) * W + iw) * C + c;
                            if (x[j] > best) { best = x[j]; at = j; }
                        }
                    }
                    if (at >= 0) dx[at] += dy[(((int64_t)n * P + p) * Q + q) * C + c];
                }
}

/* pooled = mean over (h,w); logits = pooled * W^T + bias; loss = mean over the
 * b samples of -log softmax(logits)[label]  (Eq. 2 with the cross-entropy loss). */
void ora_head_fwd(const double *a, int32_t b, int32_t H, int32_t W, int32_t C, const double *Wfc,
                  const double *bias, int32_t ncls, const int32_t *labels, double *logits, double *loss)
{
    double total = 0.0;
    for (int32_t n = 0; n < b; ++n) {
        double *lg = &logits[(int64_t)n * ncls];
        for (int32_t j = 0; j < ncls; ++j) lg[j] = bias[j];
        for (int32_t c = 0; c < C; ++c) {
            double s = 0.0;
            for (int32_t i = 0; i < H * W; ++i) s += a[((int64_t)n * H * W + i) * C + c];
            double pooled = s / (double)(H * W);
            for (int32_t j = 0; j < ncls; ++j) lg[j] += pooled * Wfc[(int64_t)j * C + c];
        }
        double mx = lg[0];
        for (int32_t j = 1; j < ncls; ++j) if (lg[j] > mx) mx = lg[j];
        double z = 0.0;
        for (int32_t j = 0; j < ncls; ++j) z += exp(lg[j] - mx);
        total += -(lg[labels[n]] - mx - log(z));
    }
    *loss = total / (double)b;
}

/* dlogits = (softmax - onehot)/b; dW = dlogits^T pooled; dbias = sum_n dlogits;
 * da[n,h,w,c] = (dlogits W)[n,c] / (H*W). */
void ora_head_bwd(const double *a, int32_t b, int32_t H, int32_t W, int32_t C, const double *Wfc,
                  int32_t ncls, const int32_t *labels, const double *logits, double *dlogits,
                  double *dW, double *dbias, double *da)
{
    for (int64_t j = 0; j < (int64_t)ncls * C; ++j) dW[j] = 0.0;
    for (int32_t j = 0; j < ncls; ++j) dbias[j] = 0.0;
    double *pooled = (double *)malloc(sizeof(double) * (size_t)C);
    for (int32_t n = 0; n < b; ++n) {
        const double *lg = &logits[(int64_t)n * ncls];
        double *dl = &dlogits[(int64_t)n * ncls];
        double mx = lg[0];
        for (int32_t j = 1; j < ncls; ++j) if (lg[j] > mx) mx = lg[j];
        double z = 0.0;
        for (int32_t j = 0; j < ncls; ++j) z += exp(lg[j] - mx);
        for (int32_t j = 0; j < ncls; ++j)
            dl[j] = (exp(lg[j] - mx) / z - (j == labels[n] ? 1.0 : 0.0)) / (double)b;
        for (int32_t c = 0; c < C; ++c) {
            double s = 0.0;
            for (int32_t i = 0; i < H * W; ++i) s += a[((int64_t)n * H * W + i) * C + c];
            pooled[c] = s / (double)(H * W);
        }
        for (int32_t j = 0; j < ncls; ++j) {
            dbias[j] += dl[j];
            for (int32_t c = 0; c < C; ++c) dW[(int64_t)j * C + c] += dl[j] * pooled[c];
        }
        for (int32_t c = 0; c < C; ++c) {
            double s = 0.0;
            for (int32_t j = 0; j < ncls; ++j) s += dl[j] * Wfc[(int64_t)j * C + c];
            for (int32_t i = 0; i < H * W; ++i) da[((int64_t)n * H * W + i) * C + c] = s / (double)(H * W);
        }
    }
    free(pooled);
}

/* Gradient accumulate/average over micro-batches (the arithmetic of the
 * gradient allreduce of Section 5.3): out = (sum_{m ascending} g_m) / M. */
void ora_grad_average(const double *g_slots, int32_t M, int64_t G, double *out)
{
    for (int64_t j = 0; j < G; ++j) {
        double s = 0.0;
        for (int32_t m = 0; m < M; ++m) s += g_slots[(int64_t)m * G + j];
        out[j] = s / (double)M;
    }
}

/* Parameter update that closes the training step (Section 5.3: after the gradient allreduce every
 * replica applies the averaged gradients, optimizer.apply_gradients()).  Stochastic gradient descent
 * with momentum in the Keras form, the framework the paper builds on:
 *     g' = g + weight_decay * theta;   v <- momentum * v - lr * g';   theta <- theta + v.
 * momentum = 0 and weight_decay = 0 give plain gradient descent theta <- theta - lr * g. */
void ora_sgd_momentum(double *theta, double *v, const double *g, int64_t G, double lr, double momentum,
                      double weight_decay)
{
    for (int64_t j = 0; j < G; ++j) {
        const double gj = g[j] + weight_decay * theta[j];
        v[j] = momentum * v[j] - lr * gj;
        theta[j] = theta[j] + v[j];
    }
}

/* ------------------------------------------------------------------ */
/* One op applied to whole tensors (used by both sweeps below)         */
/* ------------------------------------------------------------------ */

typedef struct {
    const ora_op *ops;
    int32_t n_ops, b;
    const int32_t *in_hwc;
    int32_t *hwc;                 /* n_ops*3 */
    int64_t *w_off, *w_cnt, *b_off, *b_cnt, G;
    const double *theta;          /* G */
    const int32_t *labels;        /* b */
    const uint8_t *const *decisions; /* per op (BNRELU entries used), or NULL */
    double tau;
    int64_t counts[2];
} ora_ctx;

static const int32_t *shape_of(const ora_ctx *c, int32_t t) { return t < 0 ? c->in_hwc : &c->hwc[3 * t]; }
static int64_t numel_of(const ora_ctx *c, int32_t t)
{
    const int32_t *s = shape_of(c, t);
    return (int64_t)c->b * s[0] * s[1] * s[2];
}

static void op_forward(const ora_ctx *c, int32_t i, const double *in0, const double *in1, double *out,
                       double *loss)
{
    const ora_op *o = &c->ops[i];
    const int32_t *s = shape_of(c, o->src0);
    const double *th = c->theta;
    switch (o->kind) {
    case ORA_CONV:
        ora_conv_fwd(in0, c->b, s[0], s[1], s[2], th + c->w_off[i], o->c_out, o->ksize, o->stride, o->pad, out);
        break;
    case ORA_BNRELU:
        ora_bnrelu_fwd(in0, (int64_t)c->b * s[0] * s[1], s[2], th + c->w_off[i], th + c->b_off[i], o->eps, out);
        break;
    case ORA_ADD: {
        int64_t n = numel_of(c, i);
        for (int64_t j = 0; j < n; ++j) out[j] = in0[j] + in1[j];
        break;
    }
    case ORA_BN:
        ora_bn_fwd(in0, (int64_t)c->b * s[0] * s[1], s[2], th + c->w_off[i], th + c->b_off[i], o->eps, out);
        break;
    case ORA_RELU:
        ora_relu_fwd(in0, numel_of(c, i), out);
        break;
    case ORA_MAXPOOL:
        ora_maxpool_fwd(in0, c->b, s[0], s[1], s[2], o->ksize, o->stride, o->pad, out);
        break;
    case ORA_HEAD:
        ora_head_fwd(in0, c->b, s[0], s[1], s[2], th + c->w_off[i], th + c->b_off[i], o->c_out, c->labels, out, loss);
        break;
    }
}

/* Backward of op i.  `dout` is dL/d(out) (for HEAD it is produced here, into
 * dout itself).  Contributions are ADDED into d0 / d1 (the gradients of the
 * sources; NULL = not wanted), weight gradients are written into g. */
static int op_backward(const ora_ctx *c, int32_t i, const double *in0, const double *out, double *dout,
                       double *d0, double *d1, double *g)
{
    const ora_op *o = &c->ops[i];
    const int32_t *s = shape_of(c, o->src0);
    const double *th = c->theta;
    int64_t n_in = numel_of(c, o->src0);
    double *tmp = NULL;
    if (o->kind != ORA_ADD) {
        tmp = (double *)malloc(sizeof(double) * (size_t)n_in);
        if (!tmp) return ORA_ENOMEM;
    }
    switch (o->kind) {
    case ORA_CONV:
        ora_conv_wgrad(in0, c->b, s[0], s[1], s[2], dout, o->c_out, o->ksize, o->stride, o->pad, g + c->w_off[i]);
        if (d0) ora_conv_dgrad(dout, c->b, s[0], s[1], s[2], th + c->w_off[i], o->c_out, o->ksize, o->stride, o->pad, tmp);
        break;
    case ORA_BNRELU:
        ora_bnrelu_bwd_dec(in0, dout, (int64_t)c->b * s[0] * s[1], s[2], th + c->w_off[i], th + c->b_off[i], o->eps,
                           c->decisions ? c->decisions[i] : NULL, c->tau, ((ora_ctx *)c)->counts,
                           tmp, g + c->w_off[i], g + c->b_off[i]);
        break;
    case ORA_ADD: {
        int64_t n = numel_of(c, i);
        if (d0) for (int64_t j = 0; j < n; ++j) d0[j] += dout[j];
        if (d1) for (int64_t j = 0; j < n; ++j) d1[j] += dout[j];
        return ORA_OK;
    }
    case ORA_BN:
        ora_bn_bwd(in0, dout, (int64_t)c->b * s[0] * s[1], s[2], th + c->w_off[i], o->eps, tmp, g + c->w_off[i], g + c->b_off[i]);
        break;
    case ORA_RELU:
        ora_relu_bwd_dec(in0, dout, n_in, c->decisions ? c->decisions[i] : NULL, c->tau, ((ora_ctx *)c)->counts, tmp);
        break;
    case ORA_MAXPOOL:
        ora_maxpool_bwd(in0, dout, c->b, s[0], s[1], s[2], o->ksize, o->stride, o->pad, tmp);
        break;
    case ORA_HEAD:
        ora_head_bwd(in0, c->b, s[0], s[1], s[2], th + c->w_off[i], o->c_out, c->labels, out, dout,
                     g + c->w_off[i], g + c->b_off[i], tmp);
        break;
    }
    if (d0) for (int64_t j = 0; j < n_in; ++j) d0[j] += tmp[j];
    free(tmp);
    return ORA_OK;
}

static int ctx_init(ora_ctx *c, const ora_op *ops, int32_t n_ops, int32_t b, const int32_t in_hwc[3],
                    const double *theta, const int32_t *labels)
{
    memset(c, 0, sizeof(*c));
    c->ops = ops; c->n_ops = n_ops; c->b = b; c->in_hwc = in_hwc; c->theta = theta; c->labels = labels;
    c->hwc = (int32_t *)malloc(sizeof(int32_t) * 3 * (size_t)n_ops);
    c->w_off = (int64_t *)malloc(sizeof(int64_t) * 4 * (size_t)n_ops);
    if (!c->hwc || !c->w_off) return ORA_ENOMEM;
    c->w_cnt = c->w_off + n_ops; c->b_off = c->w_cnt + n_ops; c->b_cnt = c->b_off + n_ops;
    if (ora_shapes(ops, n_ops, in_hwc, c->hwc)) return ORA_EINVAL;
    ora_param_layout(ops, n_ops, c->w_off, c->w_cnt, c->b_off, c->b_cnt, &c->G);
    for (int32_t n = 0; n < b; ++n)
        if (labels[n] < 0 || labels[n] >= ops[n_ops - 1].c_out) return ORA_EINVAL;
    return ORA_OK;
}
static void ctx_free(ora_ctx *c) { free(c->hwc); free(c->w_off); }

/* ------------------------------------------------------------------ */
/* One micro-batch, whole network in one address space                 */
/* ------------------------------------------------------------------ */

/* Forward sweep in list order, reverse sweep in descending order.
 * keep_act[i] / keep_dact[i] (either array may be NULL, any entry may be NULL)
 * receive op i's output and dL_m/d(output).  dx_in (may be NULL) receives
 * dL_m/d(network input).  g (length G) receives dL_m/d(theta). */
int ora_microbatch_dec(const ora_op *ops, int32_t n_ops, int32_t b, const int32_t in_hwc[3],
                       const double *theta, const double *x, const int32_t *labels,
                       const uint8_t *const *decisions, double tau, int64_t *counts_out,
                       double **keep_act, double **keep_dact, double *dx_in, double *g, double *loss)
{
    ora_ctx c;
    int rc = ctx_init(&c, ops, n_ops, b, in_hwc, theta, labels);
    if (rc) { ctx_free(&c); return rc; }
    c.decisions = decisions; c.tau = tau;
    double **act = (double **)calloc((size_t)n_ops, sizeof(double *));
    double **dact = (double **)calloc((size_t)n_ops, sizeof(double *));
    double *dx0 = NULL;
    for (int32_t i = 0; i < n_ops; ++i) {
        act[i] = (double *)malloc(sizeof(double) * (size_t)numel_of(&c, i));
        if (!act[i]) { rc = ORA_ENOMEM; goto done; }
        const ora_op *o = &ops[i];
        const double *in0 = o->src0 < 0 ? x : act[o->src0];
        const double *in1 = o->kind == ORA_ADD ? (o->src1 < 0 ? x : act[o->src1]) : NULL;
        op_forward(&c, i, in0, in1, act[i], loss);
        if (keep_act && keep_act[i]) memcpy(keep_act[i], act[i], sizeof(double) * (size_t)numel_of(&c, i));
    }
    for (int64_t j = 0; j < c.G; ++j) g[j] = 0.0;
    dx0 = (double *)calloc((size_t)numel_of(&c, -1), sizeof(double));
    for (int32_t i = 0; i < n_ops; ++i) {
        dact[i] = (double *)calloc((size_t)numel_of(&c, i), sizeof(double));
        if (!dact[i]) { rc = ORA_ENOMEM; goto done; }
    }
    for (int32_t i = n_ops - 1; i >= 0; --i) {
        const ora_op *o = &ops[i];
        const double *in0 = o->src0 < 0 ? x : act[o->src0];
        double *d0 = o->src0 < 0 ? dx0 : dact[o->src0];
        double *d1 = o->kind == ORA_ADD ? (o->src1 < 0 ? dx0 : dact[o->src1]) : NULL;
        rc = op_backward(&c, i, in0, act[i], dact[i], d0, d1, g);
        if (rc) goto done;
        if (keep_dact && keep_dact[i]) memcpy(keep_dact[i], dact[i], sizeof(double) * (size_t)numel_of(&c, i));
        free(dact[i]); dact[i] = NULL;   /* every consumer of op i has a larger index */
    }
    if (dx_in) memcpy(dx_in, dx0, sizeof(double) * (size_t)numel_of(&c, -1));
    if (counts_out) { counts_out[0] = c.counts[0]; counts_out[1] = c.counts[1]; }
done:
    for (int32_t i = 0; i < n_ops; ++i) { free(act[i]); free(dact[i]); }
    free(act); free(dact); free(dx0);
    ctx_free(&c);
    return rc;
}

int ora_microbatch(const ora_op *ops, int32_t n_ops, int32_t b, const int32_t in_hwc[3],
                   const double *theta, const double *x, const int32_t *labels,
                   double **keep_act, double **keep_dact, double *dx_in, double *g, double *loss)
{
    return ora_microbatch_dec(ops, n_ops, b, in_hwc, theta, x, labels, NULL, 0.0, NULL, keep_act, keep_dact, dx_in, g, loss);
}

/* ------------------------------------------------------------------ */
/* One micro-batch, partition by partition through mailboxes           */
/* ------------------------------------------------------------------ */

/* Each partition holds only the outputs of its own ops plus private copies of
 * what it received.  fwd_box[cut][j] is the message carrying the j-th live
 * tensor of that cut forward ("partial predictions"), bwd_box[cut][j] the
 * message carrying its partial error e_cut[T] = sum over consumers at or
 * after the cut of dL/dT back (Eq. 7).  A tensor that is live at two
 * successive cuts is relayed by the partition in between.
 *
 * keep_fwd / keep_bwd: optional [n_cuts][max_live] arrays of output buffers
 * for the messages; the rest as in ora_microbatch. */
int ora_microbatch_partitioned_dec(const ora_op *ops, int32_t n_ops, int32_t b, const int32_t in_hwc[3],
                                   const int32_t *cuts, int32_t n_cuts, int32_t max_live,
                                   const double *theta, const double *x, const int32_t *labels,
                                   const uint8_t *const *decisions, double tau, int64_t *counts_out,
                                   double **keep_act, double **keep_dact,
                                   double **keep_fwd, double **keep_bwd,
                                   double *g, double *loss)
{
    if (ora_check_cuts(n_ops, cuts, n_cuts)) return ORA_EINVAL;
    ora_ctx c;
    int rc = ctx_init(&c, ops, n_ops, b, in_hwc, theta, labels);
    if (rc) { ctx_free(&c); return rc; }
    c.decisions = decisions; c.tau = tau;
    int32_t P = n_cuts + 1;
    /* bounds of partition p: [lo(p), hi(p)) */
#define LO(p) ((p) == 0 ? 0 : cuts[(p) - 1])
#define HI(p) ((p) == P - 1 ? n_ops : cuts[(p)])
    int32_t *live = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_cuts + 1) * (size_t)n_ops);
    int32_t *nlive = (int32_t *)calloc((size_t)n_cuts + 1, sizeof(int32_t));
    double **fwd_box = (double **)calloc((size_t)(n_cuts + 1) * (size_t)n_ops, sizeof(double *));
    double **bwd_box = (double **)calloc((size_t)(n_cuts + 1) * (size_t)n_ops, sizeof(double *));
    /* per-partition private storage, indexed by tensor id */
    double **loc = (double **)calloc((size_t)P * (size_t)n_ops, sizeof(double *));
    for (int32_t j = 0; j < n_cuts; ++j) {
        ora_live_set(ops, n_ops, cuts[j], &live[(size_t)j * n_ops], &nlive[j]);
        if (nlive[j] > max_live && (keep_fwd || keep_bwd)) { rc = ORA_EINVAL; goto done; }
    }
    /* the network input may only be read by the first partition */
    for (int32_t i = LO(1 < P ? 1 : 0); P > 1 && i < n_ops; ++i)
        if (ops[i].src0 < 0 || (ops[i].kind == ORA_ADD && ops[i].src1 < 0)) { rc = ORA_EINVAL; goto done; }

    /* ---- forward, partition 0 first ---- */
    for (int32_t p = 0; p < P; ++p) {
        double **mine = &loc[(size_t)p * n_ops];
        if (p > 0)                                   /* recv */
            for (int32_t j = 0; j < nlive[p - 1]; ++j) {
                int32_t t = live[(size_t)(p - 1) * n_ops + j];
                size_t bytes = sizeof(double) * (size_t)numel_of(&c, t);
                mine[t] = (double *)malloc(bytes);
                memcpy(mine[t], fwd_box[(size_t)(p - 1) * n_ops + j], bytes);
            }
        for (int32_t i = LO(p); i < HI(p); ++i) {
            const ora_op *o = &ops[i];
            mine[i] = (double *)malloc(sizeof(double) * (size_t)numel_of(&c, i));
            const double *in0 = o->src0 < 0 ? x : mine[o->src0];
            const double *in1 = o->kind == ORA_ADD ? (o->src1 < 0 ? x : mine[o->src1]) : NULL;
            op_forward(&c, i, in0, in1, mine[i], loss);
            if (keep_act && keep_act[i]) memcpy(keep_act[i], mine[i], sizeof(double) * (size_t)numel_of(&c, i));
        }
        if (p < P - 1)                               /* send */
            for (int32_t j = 0; j < nlive[p]; ++j) {
                int32_t t = live[(size_t)p * n_ops + j];
                size_t bytes = sizeof(double) * (size_t)numel_of(&c, t);
                double *msg = (double *)malloc(bytes);
                memcpy(msg, mine[t], bytes);
                fwd_box[(size_t)p * n_ops + j] = msg;
                if (keep_fwd && keep_fwd[(size_t)p * max_live + j]) memcpy(keep_fwd[(size_t)p * max_live + j], msg, bytes);
            }
    }
    /* ---- backward, last partition first ---- */
    for (int64_t j = 0; j < c.G; ++j) g[j] = 0.0;
    for (int32_t p = P - 1; p >= 0; --p) {
        double **mine = &loc[(size_t)p * n_ops];
        double **dl = (double **)calloc((size_t)n_ops, sizeof(double *));
        /* gradient buffers for own outputs and for received tensors */
        for (int32_t i = LO(p); i < HI(p); ++i) dl[i] = (double *)calloc((size_t)numel_of(&c, i), sizeof(double));
        if (p > 0)
            for (int32_t j = 0; j < nlive[p - 1]; ++j) {
                int32_t t = live[(size_t)(p - 1) * n_ops + j];
                dl[t] = (double *)calloc((size_t)numel_of(&c, t), sizeof(double));
            }
        if (p < P - 1)                               /* recv partial errors */
            for (int32_t j = 0; j < nlive[p]; ++j) {
                int32_t t = live[(size_t)p * n_ops + j];
                int64_t n = numel_of(&c, t);
                const double *msg = bwd_box[(size_t)p * n_ops + j];
                for (int64_t q = 0; q < n; ++q) dl[t][q] += msg[q];
            }
        for (int32_t i = HI(p) - 1; i >= LO(p); --i) {
            const ora_op *o = &ops[i];
            const double *in0 = o->src0 < 0 ? x : mine[o->src0];
            double *d0 = o->src0 < 0 ? NULL : dl[o->src0];
            double *d1 = o->kind == ORA_ADD ? (o->src1 < 0 ? NULL : dl[o->src1]) : NULL;
            rc = op_backward(&c, i, in0, mine[i], dl[i], d0, d1, g);
            if (rc) { free(dl); goto done; }
            if (keep_dact && keep_dact[i]) memcpy(keep_dact[i], dl[i], sizeof(double) * (size_t)numel_of(&c, i));
        }
        if (p > 0)                                   /* send partial errors */
            for (int32_t j = 0; j < nlive[p - 1]; ++j) {
                int32_t t = live[(size_t)(p - 1) * n_ops + j];
                size_t bytes = sizeof(double) * (size_t)numel_of(&c, t);
                double *msg = (double *)malloc(bytes);
                memcpy(msg, dl[t], bytes);
                bwd_box[(size_t)(p - 1) * n_ops + j] = msg;
                if (keep_bwd && keep_bwd[(size_t)(p - 1) * max_live + j]) memcpy(keep_bwd[(size_t)(p - 1) * max_live + j], msg, bytes);
            }
        for (int32_t i = 0; i < n_ops; ++i) free(dl[i]);
        free(dl);
    }
    if (counts_out) { counts_out[0] = c.counts[0]; counts_out[1] = c.counts[1]; }
done:
    for (size_t j = 0; j < (size_t)(n_cuts + 1) * (size_t)n_ops; ++j) { free(fwd_box[j]); free(bwd_box[j]); }
    for (size_t j = 0; j < (size_t)P * (size_t)n_ops; ++j) free(loc[j]);
    free(fwd_box); free(bwd_box); free(loc); free(live); free(nlive);
    ctx_free(&c);
    return rc;
#undef LO
#undef HI
}

int ora_microbatch_partitioned(const ora_op *ops, int32_t n_ops, int32_t b, const int32_t in_hwc[3],
                               const int32_t *cuts, int32_t n_cuts, int32_t max_live,
                               const double *theta, const double *x, const int32_t *labels,
                               double **keep_act, double **keep_dact,
                               double **keep_fwd, double **keep_bwd,
                               double *g, double *loss)
{
    return ora_microbatch_partitioned_dec(ops, n_ops, b, in_hwc, cuts, n_cuts, max_live, theta, x, labels, NULL, 0.0,
                                          NULL, keep_act, keep_dact, keep_fwd, keep_bwd, g, loss);
}

/* ------------------------------------------------------------------ */
/* The whole step: M micro-batches, gradient slots, average            */
/* ------------------------------------------------------------------ */

/* x: [B][H][W][C]; labels: [B]; g_slots: [M][G]; g_avg: [G]; losses: [M].
 * n_cuts < 0 selects the single-address-space sweep. */
int ora_step(const ora_op *ops, int32_t n_ops, int32_t B, const int32_t in_hwc[3],
             const int32_t *cuts, int32_t n_cuts, int32_t M,
             const double *theta, const double *x, const int32_t *labels,
             double *g_slots, double *g_avg, double *losses, double *loss)
{
    int32_t first, end;
    if (ora_microbatch_range(B, M, 0, &first, &end)) return ORA_EINVAL;
    int32_t b = B / M;
    int64_t per = (int64_t)in_hwc[0] * in_hwc[1] * in_hwc[2];
    int64_t *lay = (int64_t *)malloc(sizeof(int64_t) * 4 * (size_t)n_ops), G;
    ora_param_layout(ops, n_ops, lay, lay + n_ops, lay + 2 * n_ops, lay + 3 * n_ops, &G);
    free(lay);
    for (int32_t m = 0; m < M; ++m) {
        ora_microbatch_range(B, M, m, &first, &end);
        int rc;
        if (n_cuts < 0)
            rc = ora_microbatch(ops, n_ops, b, in_hwc, theta, x + (int64_t)first * per, labels + first,
                                NULL, NULL, NULL, g_slots + (int64_t)m * G, &losses[m]);
        else
            rc = ora_microbatch_partitioned(ops, n_ops, b, in_hwc, cuts, n_cuts, 0, theta,
                                            x + (int64_t)first * per, labels + first,
                                            NULL, NULL, NULL, NULL, g_slots + (int64_t)m * G, &losses[m]);
        if (rc) return rc;
    }
    ora_grad_average(g_slots, M, G, g_avg);
    double s = 0.0;
    for (int32_t m = 0; m < M; ++m) s += losses[m];
    *loss = s / (double)M;
    return ORA_OK;
}
