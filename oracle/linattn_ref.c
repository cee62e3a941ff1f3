/*
 * fp64 CPU oracle for non-causal linear attention with the Hedgehog feature map.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of the
 * operator that the CUDA library is checked against.  It shares no code with
 * the CUDA path and the product never calls it: only the tests, the smoke check
 * and the benchmark's CPU-baseline leg may load it.
 *
 * What it computes, for every group g = (batch, head) independently:
 *
 *   Eq. 6   phi(x) = softmax(x W) (+) softmax(-x W)      W is d x d/2, (+) = concat,
 *                                                        softmax over the d/2 features
 *   Eq. 5   o_i = sum_j  a_ij / (sum_j a_ij) * v_j ,     a_ij = phi(q_i) . phi(k_j)   (left form)
 *           o_i = phi(q_i) S / (phi(q_i) . z) ,          S = sum_j phi(k_j)^T v_j,
 *                                                        z = sum_j phi(k_j)           (right form)
 *
 * ref_quadratic is the left form written out (the plain definition, O(n^2 d));
 * ref_linear is the right form.  Their agreement is the identity of Eq. 5 and is
 * one of the pins in the CPU tests.
 *
 *   Eq. 8   o_i = r^ * softmax-attention_i + (1 - r^) * linear-attention_i,  r^ = clip(r, 0, 1)
 *
 * ref_softmax is the first term (Eq. 4 with sim = exp) and ref_mix the blend; both at the
 * end of the file.
 *
 * Readings taken where the paper says nothing:
 *   - d is the per-head dimension; one W_q and one W_k per head (or one shared by
 *     all heads when per_head == 0).
 *   - no bias, temperature, 1/sqrt(d) scale or epsilon anywhere in the operator.
 *   - concat order is [softmax(+u), softmax(-u)].
 *   - each softmax subtracts its row maximum first (mathematically a no-op).
 *   - no mask: every one of the n tokens attends to every one of the n tokens.
 *
 * Inputs are float (already rounded to whatever storage type the GPU receives:
 * every bf16 value is exactly a float) and are widened to double on first use.
 * All sums are sequential in index order, in double.
 *
 * Threading: OpenMP over groups (state pass) and over (group, query row) (output
 * pass).  No reduction crosses threads, so results do not depend on thread count.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Eq. 6 for one row x[0..d) with W[d][m] row-major, m = d/2.  phi has d entries. */
static void phi_row(const float *x, const float *W, int d, double *phi)
{
    const int m = d / 2;
    double *u = phi + m; /* logits parked in the second half until it is overwritten */
    for (int j = 0; j < m; ++j) {
        double acc = 0.0;
        for (int c = 0; c < d; ++c)
            acc += (double)x[c] * (double)W[(size_t)c * m + j];
        u[j] = acc;
    }
    double umax = u[0], umin = u[0];
    for (int j = 1; j < m; ++j) {
        if (u[j] > umax) umax = u[j];
        if (u[j] < umin) umin = u[j];
    }
    /* softmax(+u): exp(u - max) / sum */
    double sp = 0.0;
    for (int j = 0; j < m; ++j) {
        phi[j] = exp(u[j] - umax);
        sp += phi[j];
    }
    for (int j = 0; j < m; ++j)
        phi[j] /= sp;
    /* softmax(-u): max of -u is -min(u), so exp(-u + min) / sum; overwrites u in place */
    double sn = 0.0;
    for (int j = 0; j < m; ++j) {
        u[j] = exp(umin - u[j]);
        sn += u[j];
    }
    for (int j = 0; j < m; ++j)
        u[j] /= sn;
}

static const float *w_of(const float *W, int g, int H, int d, int per_head)
{
    return per_head ? W + (size_t)(g % H) * d * (d / 2) : W;
}

/* number of threads an OpenMP region would use here (1 without OpenMP) */
int linattn_ref_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Eq. 6 applied to n rows: phi_out[n][d]. */
int linattn_ref_phi(const float *x, const float *W, long n, int d, double *phi_out)
{
    if (d < 2 || d > 4096 || (d & 1) || n < 0) return 1;
    for (long i = 0; i < n; ++i)
        phi_row(x + (size_t)i * d, W, d, phi_out + (size_t)i * d);
    return 0;
}

/*
 * Left form of Eq. 5.
 *   q,k,v : [G][n][d] float, G = B*H groups, group g uses head g % H
 *   Wq,Wk : [H][d][d/2] (per_head != 0) or [d][d/2]
 *   rows  : nrows query indices in [0,n) evaluated in every group, or NULL for all n
 *   out   : [G][nrows or n][d] double
 */
int linattn_ref_quadratic(const float *q, const float *k, const float *v,
                          const float *Wq, const float *Wk,
                          long G, int H, long n, int d, int per_head,
                          const long *rows, long nrows, double *out)
{
    if (d < 2 || d > 4096 || (d & 1) || n < 1 || G < 1 || H < 1) return 1;
    const long nr = rows ? nrows : n;
    int fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (long g = 0; g < G; ++g) {
        double *phik = (double *)malloc((size_t)n * d * sizeof(double));
        double *a = (double *)malloc((size_t)n * sizeof(double));
        double *phiq = (double *)malloc((size_t)d * sizeof(double));
        if (!phik || !a || !phiq) {
            fail = 1;
        } else {
            const float *kg = k + (size_t)g * n * d, *vg = v + (size_t)g * n * d;
            const float *qg = q + (size_t)g * n * d;
            for (long j = 0; j < n; ++j)
                phi_row(kg + (size_t)j * d, w_of(Wk, (int)g, H, d, per_head), d, phik + (size_t)j * d);
            for (long r = 0; r < nr; ++r) {
                const long i = rows ? rows[r] : r;
                double *o = out + ((size_t)g * nr + r) * d;
                phi_row(qg + (size_t)i * d, w_of(Wq, (int)g, H, d, per_head), d, phiq);
                double den = 0.0;
                for (long j = 0; j < n; ++j) {
                    double s = 0.0;
                    for (int f = 0; f < d; ++f)
                        s += phiq[f] * phik[(size_t)j * d + f];
                    a[j] = s;
                    den += s;
                }
                for (int c = 0; c < d; ++c) o[c] = 0.0;
                for (long j = 0; j < n; ++j) {
                    const double w = a[j] / den;
                    for (int c = 0; c < d; ++c)
                        o[c] += w * (double)vg[(size_t)j * d + c];
                }
            }
        }
        free(phik); free(a); free(phiq);
    }
    return fail;
}

/*
 * Right form of Eq. 5.  Arguments as above, plus optional state outputs
 *   S_out : [G][d][d] double, S[f][c] = sum_j phi(k_j)[f] * v_j[c]   (may be NULL)
 *   z_out : [G][d]    double, z[f]    = sum_j phi(k_j)[f]            (may be NULL)
 * out may be NULL when only the state is wanted.
 */
int linattn_ref_linear(const float *q, const float *k, const float *v,
                       const float *Wq, const float *Wk,
                       long G, int H, long n, int d, int per_head,
                       const long *rows, long nrows, double *out,
                       double *S_out, double *z_out)
{
    if (d < 2 || d > 4096 || (d & 1) || n < 1 || G < 1 || H < 1) return 1;
    const long nr = rows ? nrows : n;
    double *S_all = (double *)calloc((size_t)G * d * d, sizeof(double));
    double *z_all = (double *)calloc((size_t)G * d, sizeof(double));
    if (!S_all || !z_all) { free(S_all); free(z_all); return 1; }

    /* state pass: S and z of every group, tokens in index order */
#pragma omp parallel for schedule(dynamic, 1)
    for (long g = 0; g < G; ++g) {
        double phik[4096]; /* d <= 4096 */
        double *S = S_all + (size_t)g * d * d, *z = z_all + (size_t)g * d;
        const float *kg = k + (size_t)g * n * d, *vg = v + (size_t)g * n * d;
        for (long j = 0; j < n; ++j) {
            phi_row(kg + (size_t)j * d, w_of(Wk, (int)g, H, d, per_head), d, phik);
            for (int f = 0; f < d; ++f) {
                z[f] += phik[f];
                for (int c = 0; c < d; ++c)
                    S[(size_t)f * d + c] += phik[f] * (double)vg[(size_t)j * d + c];
            }
        }
    }

    /* output pass: o_i = phi(q_i) S / (phi(q_i) . z) */
    if (out) {
#pragma omp parallel for collapse(2) schedule(static)
        for (long g = 0; g < G; ++g) {
            for (long r = 0; r < nr; ++r) {
                double phiq[4096];
                const long i = rows ? rows[r] : r;
                const double *S = S_all + (size_t)g * d * d, *z = z_all + (size_t)g * d;
                double *o = out + ((size_t)g * nr + r) * d;
                phi_row(q + ((size_t)g * n + i) * d, w_of(Wq, (int)g, H, d, per_head), d, phiq);
                double den = 0.0;
                for (int f = 0; f < d; ++f)
                    den += phiq[f] * z[f];
                for (int c = 0; c < d; ++c) {
                    double num = 0.0;
                    for (int f = 0; f < d; ++f)
                        num += phiq[f] * S[(size_t)f * d + c];
                    o[c] = num / den;
                }
            }
        }
    }
    if (S_out) memcpy(S_out, S_all, (size_t)G * d * d * sizeof(double));
    if (z_out) memcpy(z_out, z_all, (size_t)G * d * sizeof(double));
    free(S_all); free(z_all);
    return 0;
}

/*
 * First term of Eq. 8 (Eq. 4 with sim = exp): softmax attention,
 *   o_i = sum_j exp(scale * q_i . k_j) v_j / sum_j exp(scale * q_i . k_j),
 * all n tokens attending to all n tokens.  The paper prints the scale as 1/sqrt(d) in the text
 * under Eq. 4 and as 1/d inside Eq. 8; it is an argument here.  The row maximum is subtracted
 * before exponentiating (mathematically a no-op).
 *   q,k,v : [G][n][d] float;  rows : nrows query indices, or NULL for all n
 *   out   : [G][nrows or n][d] double
 */
int linattn_ref_softmax(const float *q, const float *k, const float *v,
                        long G, long n, int d, double scale,
                        const long *rows, long nrows, double *out)
{
    if (d < 1 || n < 1 || G < 1) return 1;
    const long nr = rows ? nrows : n;
    int fail = 0;
#pragma omp parallel for schedule(dynamic, 8) collapse(2)
    for (long g = 0; g < G; ++g) {
        for (long r = 0; r < nr; ++r) {
            double *s = (double *)malloc((size_t)n * sizeof(double));
            if (!s) {
                fail = 1;
                continue;
            }
            const long i = rows ? rows[r] : r;
            const float *qi = q + ((size_t)g * n + i) * d;
            const float *kg = k + (size_t)g * n * d, *vg = v + (size_t)g * n * d;
            double smax = 0.0;
            for (long j = 0; j < n; ++j) {
                double acc = 0.0;
                for (int c = 0; c < d; ++c) acc += (double)qi[c] * (double)kg[(size_t)j * d + c];
                s[j] = scale * acc;
                if (j == 0 || s[j] > smax) smax = s[j];
            }
            double den = 0.0;
            for (long j = 0; j < n; ++j) {
                s[j] = exp(s[j] - smax);
                den += s[j];
            }
            double *o = out + ((size_t)g * nr + r) * d;
            for (int c = 0; c < d; ++c) o[c] = 0.0;
            for (long j = 0; j < n; ++j) {
                const double w = s[j] / den;
                for (int c = 0; c < d; ++c) o[c] += w * (double)vg[(size_t)j * d + c];
            }
            free(s);
        }
    }
    return fail;
}

/*
 * Eq. 8: out = r^ * o_softmax + (1 - r^) * o_linear, element by element, with the learnable
 * score r clipped into [0, 1] first (footnote to Eq. 8): r^ = min(max(r, 0), 1).
 */
int linattn_ref_mix(const double *o_softmax, const double *o_linear, long count, double r, double *out)
{
    if (count < 0) return 1;
    const double rc = r < 0.0 ? 0.0 : (r > 1.0 ? 1.0 : r);
    for (long e = 0; e < count; ++e) out[e] = rc * o_softmax[e] + (1.0 - rc) * o_linear[e];
    return 0;
}

/*
 * Gradients of the operator (what the post-training objective of Eq. 14 back-propagates through every
 * linear-attention layer): for L = sum_{i,c} dO[i][c] * o_i[c] with o from the right form of Eq. 5 and
 * phi from Eq. 6, the derivatives of L with respect to q, k, v, W_q and W_k, by the chain rule written out:
 *
 *   dnum_i = dO_i / den_i                      dden_i = -(dO_i . o_i) / den_i
 *   dphi(q_i) = S dnum_i + dden_i z            dS = sum_i phi(q_i)^T dnum_i        dz = sum_i dden_i phi(q_i)
 *   dphi(k_j) = dS v_j + dz                    dv_j = dS^T phi(k_j)
 *   through phi (two softmaxes p+ = softmax(u), p- = softmax(-u), u = x W):
 *       du = p+ (.) (dphi+ - p+ . dphi+)  -  p- (.) (dphi- - p- . dphi-)
 *       dx = du W^T                            dW += x^T du
 *
 * dW_q, dW_k are summed over the batch (groups g with the same head g % H) and, when per_head == 0, over the
 * heads as well.  All arrays [G][n][d] except dWq, dWk: [H][d][d/2] (per_head) or [d][d/2].  Outputs in double.
 */
static void phi_backward_row(const float *x, const float *W, int d, const double *phi, const double *dphi,
                             double *dx, double *dW)
{
    const int m = d / 2;
    double dotp = 0.0, dotn = 0.0;
    for (int j = 0; j < m; ++j) {
        dotp += phi[j] * dphi[j];
        dotn += phi[m + j] * dphi[m + j];
    }
    for (int c = 0; c < d; ++c) dx[c] = 0.0;
    for (int j = 0; j < m; ++j) {
        const double du = phi[j] * (dphi[j] - dotp) - phi[m + j] * (dphi[m + j] - dotn);
        for (int c = 0; c < d; ++c) {
            dx[c] += du * (double)W[(size_t)c * m + j];
            dW[(size_t)c * m + j] += (double)x[c] * du;
        }
    }
}

/* The chain rule above for an incoming gradient lin_scale * dout (lin_scale = 1 for the plain operator; Eq. 8 hands the
 * linear branch (1 - r^) times the layer's gradient).  *sum_dout_o, if not NULL, receives sum_{g,i,c} dout * o with the
 * UNSCALED dout: the part of dL/dr that comes from the linear branch. */
static int backward_core(const float *q, const float *k, const float *v, const float *Wq, const float *Wk,
                         const float *dout, double lin_scale, long G, int H, long n, int d, int per_head,
                         double *dq, double *dk, double *dv, double *dWq, double *dWk, double *sum_dout_o)
{
    if (d < 2 || d > 4096 || (d & 1) || n < 1 || G < 1 || H < 1) return 1;
    const int m = d / 2;
    const size_t wsz = (size_t)d * m;
    const long nW = per_head ? H : 1;
    for (size_t e = 0; e < (size_t)nW * wsz; ++e) dWq[e] = dWk[e] = 0.0;
    int fail = 0;
    /* one group at a time (the weight gradients are shared between groups, so no threading across groups) */
    for (long g = 0; g < G && !fail; ++g) {
        const float *qg = q + (size_t)g * n * d, *kg = k + (size_t)g * n * d, *vg = v + (size_t)g * n * d;
        const float *gg = dout + (size_t)g * n * d;
        const float *wq = w_of(Wq, (int)g, H, d, per_head), *wk = w_of(Wk, (int)g, H, d, per_head);
        double *dwq = dWq + (per_head ? (size_t)(g % H) * wsz : 0), *dwk = dWk + (per_head ? (size_t)(g % H) * wsz : 0);
        double *S = (double *)calloc((size_t)d * d, sizeof(double)), *z = (double *)calloc(d, sizeof(double));
        double *dS = (double *)calloc((size_t)d * d, sizeof(double)), *dz = (double *)calloc(d, sizeof(double));
        double *phi = (double *)malloc((size_t)d * sizeof(double)), *dphi = (double *)malloc((size_t)d * sizeof(double));
        double *o = (double *)malloc((size_t)d * sizeof(double)), *dnum = (double *)malloc((size_t)d * sizeof(double));
        if (!S || !z || !dS || !dz || !phi || !dphi || !o || !dnum) {
            fail = 1;
        } else {
            /* forward state */
            for (long j = 0; j < n; ++j) {
                phi_row(kg + (size_t)j * d, wk, d, phi);
                for (int f = 0; f < d; ++f) {
                    z[f] += phi[f];
                    for (int c = 0; c < d; ++c) S[(size_t)f * d + c] += phi[f] * (double)vg[(size_t)j * d + c];
                }
            }
            /* query side: dq, dWq, and the gradients of the state */
            for (long i = 0; i < n; ++i) {
                phi_row(qg + (size_t)i * d, wq, d, phi);
                double den = 0.0;
                for (int f = 0; f < d; ++f) den += phi[f] * z[f];
                double go = 0.0;
                for (int c = 0; c < d; ++c) {
                    double num = 0.0;
                    for (int f = 0; f < d; ++f) num += phi[f] * S[(size_t)f * d + c];
                    o[c] = num / den;
                    const double gin = lin_scale * (double)gg[(size_t)i * d + c];   /* gradient that reaches the linear branch */
                    go += gin * o[c];
                    dnum[c] = gin / den;
                    if (sum_dout_o) *sum_dout_o += (double)gg[(size_t)i * d + c] * o[c];
                }
                const double dden = -go / den;
                for (int f = 0; f < d; ++f) {
                    double acc = dden * z[f];
                    for (int c = 0; c < d; ++c) {
                        acc += S[(size_t)f * d + c] * dnum[c];
                        dS[(size_t)f * d + c] += phi[f] * dnum[c];
                    }
                    dphi[f] = acc;
                    dz[f] += dden * phi[f];
                }
                phi_backward_row(qg + (size_t)i * d, wq, d, phi, dphi, dq + ((size_t)g * n + i) * d, dwq);
            }
            /* key side: dk, dv, dWk */
            for (long j = 0; j < n; ++j) {
                phi_row(kg + (size_t)j * d, wk, d, phi);
                double *dvj = dv + ((size_t)g * n + j) * d;
                for (int c = 0; c < d; ++c) dvj[c] = 0.0;
                for (int f = 0; f < d; ++f) {
                    double acc = dz[f];
                    for (int c = 0; c < d; ++c) {
                        acc += dS[(size_t)f * d + c] * (double)vg[(size_t)j * d + c];
                        dvj[c] += phi[f] * dS[(size_t)f * d + c];
                    }
                    dphi[f] = acc;
                }
                phi_backward_row(kg + (size_t)j * d, wk, d, phi, dphi, dk + ((size_t)g * n + j) * d, dwk);
            }
        }
        free(S); free(z); free(dS); free(dz); free(phi); free(dphi); free(o); free(dnum);
    }
    return fail;
}

int linattn_ref_backward(const float *q, const float *k, const float *v, const float *Wq, const float *Wk,
                         const float *dout, long G, int H, long n, int d, int per_head,
                         double *dq, double *dk, double *dv, double *dWq, double *dWk)
{
    return backward_core(q, k, v, Wq, Wk, dout, 1.0, G, H, n, d, per_head, dq, dk, dv, dWq, dWk, NULL);
}

/*
 * Gradients through the mixed attention of Eq. 8,  out = r^ * a + (1 - r^) * lin(q, k, v),  r^ = clip(r, 0, 1), where a
 * is the output of the softmax-attention branch (given) and lin the operator of Eq. 5 / Eq. 6.  For L = sum dout * out:
 *
 *   dL/da     = r^ * dout
 *   dL/dlin   = (1 - r^) * dout      -> dq, dk, dv, dW_q, dW_k by the chain rule above with that incoming gradient
 *   dL/dr     = sum dout * (a - lin)  if 0 <= r <= 1,  else 0
 *
 * Reading taken for the clip (the paper's footnote to Eq. 8 clips r into [0, 1] and says nothing of its derivative): the
 * derivative of clip is 1 on the closed interval, ends included, and 0 outside.  The ends must be included for the
 * method to work at all: the paper initialises every r to 1, and with a zero derivative at r = 1 no score could ever
 * leave its initial value.  da may be NULL.  a: [G][n][d] float; dr: one double.
 */
int linattn_ref_backward_mixed(const float *q, const float *k, const float *v, const float *Wq, const float *Wk,
                               const float *a, double r, const float *dout, long G, int H, long n, int d, int per_head,
                               double *dq, double *dk, double *dv, double *dWq, double *dWk, double *da, double *dr)
{
    if (!dr || r != r) return 1;
    const double rc = r < 0.0 ? 0.0 : (r > 1.0 ? 1.0 : r);
    double sum_dout_o = 0.0;
    if (backward_core(q, k, v, Wq, Wk, dout, 1.0 - rc, G, H, n, d, per_head, dq, dk, dv, dWq, dWk, &sum_dout_o)) return 1;
    double sum_dout_a = 0.0;
    for (size_t e = 0; e < (size_t)G * n * d; ++e) {
        sum_dout_a += (double)dout[e] * (double)a[e];
        if (da) da[e] = rc * (double)dout[e];
    }
    *dr = (r >= 0.0 && r <= 1.0) ? sum_dout_a - sum_dout_o : 0.0;
    return 0;
}

/*
 * The ReLU kernel function of the paper's ablation over kernel functions (the table "Comparison across kernel
 * functions"; the paper names the kernel and prints no formula).  Reading taken: the standard ReLU feature map of
 * the linear-attention literature the ablation follows, phi(x) = max(x, 0) element by element on the d features of
 * the head, no learnable matrix; Eq. 5 is otherwise unchanged (no epsilon: a query whose phi is orthogonal to z
 * divides by zero and gives a non-finite row, on both sides).  Left and right forms as for the Hedgehog map.
 *   q,k,v : [G][n][d] float;  rows : nrows query indices, or NULL for all n;  out : [G][nrows or n][d] double
 */
static double relu(float x) { return x > 0.0f ? (double)x : 0.0; }

int linattn_ref_relu_quadratic(const float *q, const float *k, const float *v, long G, long n, int d,
                               const long *rows, long nrows, double *out)
{
    if (d < 1 || n < 1 || G < 1) return 1;
    const long nr = rows ? nrows : n;
    int fail = 0;
#pragma omp parallel for collapse(2) schedule(static)
    for (long g = 0; g < G; ++g) {
        for (long r = 0; r < nr; ++r) {
            const long i = rows ? rows[r] : r;
            const float *qi = q + ((size_t)g * n + i) * d;
            const float *kg = k + (size_t)g * n * d, *vg = v + (size_t)g * n * d;
            double *o = out + ((size_t)g * nr + r) * d;
            double *a = (double *)malloc((size_t)n * sizeof(double));
            if (!a) { fail = 1; continue; }
            double den = 0.0;
            for (long j = 0; j < n; ++j) {
                double s = 0.0;
                for (int f = 0; f < d; ++f) s += relu(qi[f]) * relu(kg[(size_t)j * d + f]);
                a[j] = s;
                den += s;
            }
            for (int c = 0; c < d; ++c) o[c] = 0.0;
            for (long j = 0; j < n; ++j)
                for (int c = 0; c < d; ++c) o[c] += a[j] / den * (double)vg[(size_t)j * d + c];
            free(a);
        }
    }
    return fail;
}

int linattn_ref_relu_linear(const float *q, const float *k, const float *v, long G, long n, int d,
                            const long *rows, long nrows, double *out, double *S_out, double *z_out)
{
    if (d < 1 || n < 1 || G < 1) return 1;
    const long nr = rows ? nrows : n;
    double *S_all = (double *)calloc((size_t)G * d * d, sizeof(double));
    double *z_all = (double *)calloc((size_t)G * d, sizeof(double));
    if (!S_all || !z_all) { free(S_all); free(z_all); return 1; }
#pragma omp parallel for schedule(dynamic, 1)
    for (long g = 0; g < G; ++g) {
        double *S = S_all + (size_t)g * d * d, *z = z_all + (size_t)g * d;
        for (long j = 0; j < n; ++j) {
            const float *kj = k + ((size_t)g * n + j) * d, *vj = v + ((size_t)g * n + j) * d;
            for (int f = 0; f < d; ++f) {
                const double p = relu(kj[f]);
                z[f] += p;
                for (int c = 0; c < d; ++c) S[(size_t)f * d + c] += p * (double)vj[c];
            }
        }
    }
    if (out) {
#pragma omp parallel for collapse(2) schedule(static)
        for (long g = 0; g < G; ++g) {
            for (long r = 0; r < nr; ++r) {
                const long i = rows ? rows[r] : r;
                const float *qi = q + ((size_t)g * n + i) * d;
                const double *S = S_all + (size_t)g * d * d, *z = z_all + (size_t)g * d;
                double *o = out + ((size_t)g * nr + r) * d;
                double den = 0.0;
                for (int f = 0; f < d; ++f) den += relu(qi[f]) * z[f];
                for (int c = 0; c < d; ++c) {
                    double num = 0.0;
                    for (int f = 0; f < d; ++f) num += relu(qi[f]) * S[(size_t)f * d + c];
                    o[c] = num / den;
                }
            }
        }
    }
    if (S_out) memcpy(S_out, S_all, (size_t)G * d * d * sizeof(double));
    if (z_out) memcpy(z_out, z_all, (size_t)G * d * sizeof(double));
    free(S_all); free(z_all);
    return 0;
}

/*
 * Gradients of Eq. 5 with the ReLU kernel function (reading above: phi(x) = max(x, 0), no weights).  The chain rule of
 * the operator is the one written out before linattn_ref_backward; only the last step differs: d phi / d x is 1 where
 * x > 0 and 0 elsewhere (at x = 0 the subgradient 0 is taken, as the automatic differentiation of max(x, 0) does), so
 *   dq_i = dphi(q_i) (.) [q_i > 0]        dk_j = dphi(k_j) (.) [k_j > 0]        dv_j = dS^T phi(k_j).
 * All arrays [G][n][d]; inputs float, outputs double.
 */
int linattn_ref_relu_backward(const float *q, const float *k, const float *v, const float *dout, long G, long n, int d,
                              double *dq, double *dk, double *dv)
{
    if (d < 1 || d > 4096 || n < 1 || G < 1) return 1;
    int fail = 0;
#pragma omp parallel for schedule(dynamic)
    for (long g = 0; g < G; ++g) {
        const float *qg = q + (size_t)g * n * d, *kg = k + (size_t)g * n * d, *vg = v + (size_t)g * n * d;
        const float *gg = dout + (size_t)g * n * d;
        double *S = (double *)calloc((size_t)d * d, sizeof(double)), *z = (double *)calloc(d, sizeof(double));
        double *dS = (double *)calloc((size_t)d * d, sizeof(double)), *dz = (double *)calloc(d, sizeof(double));
        double *o = (double *)malloc((size_t)d * sizeof(double)), *dnum = (double *)malloc((size_t)d * sizeof(double));
        if (!S || !z || !dS || !dz || !o || !dnum) {
            fail = 1;
        } else {
            for (long j = 0; j < n; ++j)
                for (int f = 0; f < d; ++f) {
                    const double pf = relu(kg[(size_t)j * d + f]);
                    z[f] += pf;
                    for (int c = 0; c < d; ++c) S[(size_t)f * d + c] += pf * (double)vg[(size_t)j * d + c];
                }
            for (long i = 0; i < n; ++i) {
                const float *qi = qg + (size_t)i * d;
                double den = 0.0;
                for (int f = 0; f < d; ++f) den += relu(qi[f]) * z[f];
                double go = 0.0;
                for (int c = 0; c < d; ++c) {
                    double num = 0.0;
                    for (int f = 0; f < d; ++f) num += relu(qi[f]) * S[(size_t)f * d + c];
                    o[c] = num / den;
                    go += (double)gg[(size_t)i * d + c] * o[c];
                    dnum[c] = (double)gg[(size_t)i * d + c] / den;
                }
                const double dden = -go / den;
                for (int f = 0; f < d; ++f) {
                    double acc = dden * z[f];
                    for (int c = 0; c < d; ++c) {
                        acc += S[(size_t)f * d + c] * dnum[c];
                        dS[(size_t)f * d + c] += relu(qi[f]) * dnum[c];
                    }
                    dz[f] += dden * relu(qi[f]);
                    dq[((size_t)g * n + i) * d + f] = qi[f] > 0.0f ? acc : 0.0;
                }
            }
            for (long j = 0; j < n; ++j) {
                const float *kj = kg + (size_t)j * d;
                double *dvj = dv + ((size_t)g * n + j) * d;
                for (int c = 0; c < d; ++c) dvj[c] = 0.0;
                for (int f = 0; f < d; ++f) {
                    double acc = dz[f];
                    for (int c = 0; c < d; ++c) {
                        acc += dS[(size_t)f * d + c] * (double)vg[(size_t)j * d + c];
                        dvj[c] += relu(kj[f]) * dS[(size_t)f * d + c];
                    }
                    dk[((size_t)g * n + j) * d + f] = kj[f] > 0.0f ? acc : 0.0;
                }
            }
        }
        free(S); free(z); free(dS); free(dz); free(o); free(dnum);
    }
    return fail;
}
