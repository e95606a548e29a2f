/*
 * gr_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, fp64 CPU restatement of the "global resolution" verification
 * rule for n i.i.d. drafts (optimal multi-draft speculative sampling).  It is
 * the yardstick the CUDA library is compared with; it shares no code with it
 * and nothing in the product path may call it.
 *
 * Letters: "tgt" is the target-model distribution (the paper's p), "drf" the
 * single-token draft distribution after temperature / top-k (the paper's q),
 * n the number of i.i.d. drafts.  Each function names the passage it follows.
 *
 * Pinning (see tests, all run without a GPU):
 *   - optimal acceptance alpha* : brute-force LP / max-flow over all V^n tuples,
 *     2^V subset enumeration, the n=1 closed form sum_x min(tgt,drf), monotone in n.
 *   - outer residuals p_i, r_i  : every Hall inequality on tiny V, the sum rules.
 *   - grouped-term gradient (route G1): tuple enumeration.
 *   - integral gradient (route G2): G1 and tuple enumeration on small supports.
 *   - block rule + softmax solves + slice: the assembled coupling has column sums
 *     drf^n(omega), row sums tgt exactly and accepted mass alpha*.
 *   - draw: integrates back to the slice.
 * At supports too large for G1 (k=50, n=8 ...) the only pins are alpha*'s closed
 * form and the G2 marginal certificate; beyond that: parity unpinned.
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fopenmp -shared -fPIC gr_oracle.c -lm
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#include <stdint.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define GRO_OK 0
#define GRO_NOT_CONVERGED 1
#define GRO_BAD_ARG (-1)
#define GRO_DRAFT_OUT_OF_SUPPORT (-2)

/* ------------------------------------------------------------------ O1, O2
 * Distributions from logits.  Temperature and top-k only change how the two
 * distributions are computed from the logits (App. A, first paragraph); top-k
 * on the draft reduces the problem to the kept ids (App. N).
 *   tgt_i = softmax(tl / Tt) over the whole vocabulary,
 *   support = the k largest draft logits (equal logits: smaller id is kept),
 *   drf_i = softmax(dl / Td) over the support, 0 elsewhere.
 * ids_out receives the support in ascending id order; returns k.
 */
typedef struct { double v; int id; } kv_t;

static int cmp_logit_desc(const void *a, const void *b)
{
    const kv_t *x = (const kv_t *)a, *y = (const kv_t *)b;
    if (x->v > y->v) return -1;
    if (x->v < y->v) return 1;
    return (x->id < y->id) ? -1 : (x->id > y->id);
}
static int cmp_int_asc(const void *a, const void *b)
{
    int x = *(const int *)a, y = *(const int *)b;
    return (x < y) ? -1 : (x > y);
}

int gro_distributions(const double *tl, const double *dl, int V, int topk,
                      double Tt, double Td, double *tgt, double *drf,
                      int *ids_out, double *lse_t_out)
{
    if (V <= 0 || Tt <= 0.0 || Td <= 0.0) return GRO_BAD_ARG;
    int k = (topk <= 0 || topk >= V) ? V : topk;
    double mx = -INFINITY;
    for (int i = 0; i < V; i++) { double a = tl[i] / Tt; if (a > mx) mx = a; }
    double s = 0.0;
    for (int i = 0; i < V; i++) s += exp(tl[i] / Tt - mx);
    double lse_t = mx + log(s);
    for (int i = 0; i < V; i++) tgt[i] = exp(tl[i] / Tt - lse_t);
    if (lse_t_out) *lse_t_out = lse_t;

    kv_t *kv = (kv_t *)malloc(sizeof(kv_t) * (size_t)V);
    for (int i = 0; i < V; i++) { kv[i].v = dl[i]; kv[i].id = i; }
    qsort(kv, (size_t)V, sizeof(kv_t), cmp_logit_desc);
    for (int j = 0; j < k; j++) ids_out[j] = kv[j].id;
    free(kv);
    qsort(ids_out, (size_t)k, sizeof(int), cmp_int_asc);

    double mb = -INFINITY;
    for (int j = 0; j < k; j++) { double b = dl[ids_out[j]] / Td; if (b > mb) mb = b; }
    double sb = 0.0;
    for (int j = 0; j < k; j++) sb += exp(dl[ids_out[j]] / Td - mb);
    double lse_d = mb + log(sb);
    for (int i = 0; i < V; i++) drf[i] = 0.0;
    for (int j = 0; j < k; j++) drf[ids_out[j]] = exp(dl[ids_out[j]] / Td - lse_d);
    return k;
}

/* ------------------------------------------------------------------ O3
 * Subset selection (Sec. 3.2, Eq. "subset-select"; Sec. 5.1): for i.i.d. drafts
 * it suffices to sort by decreasing drf/tgt and take the prefix minimising
 *   psi(H) = tgt(H) - drf(H)^n ;   alpha* = 1 + min psi.
 * The order is taken on the log-ratio up to its common constant,
 *   key_i = dl_i/Td - tl_i/Tt   (IEEE fp64 division and subtraction, no fusing),
 * equal keys: smaller id first.  Several minimisers: the shortest prefix.
 * The last prefix is the whole support, whose draft mass is 1 by normalisation
 * (and whose target mass is 1 too when nothing was truncated): those closing
 * values are set exactly, so that psi(V) = 0 ties with psi(empty) instead of
 * differing from it by rounding noise.
 * order_out[j] = token id at position j; psi_out has k+1 entries (psi_0 = 0).
 */
static int cmp_key_desc(const void *a, const void *b) { return cmp_logit_desc(a, b); }

int gro_subset_selection(const double *tl, const double *dl, const double *tgt,
                         const double *drf, const int *ids, int k, int n,
                         double Tt, double Td, int full_support, int *order_out, double *psi_out,
                         double *Tg_out, double *Dr_out, double *alpha_star_out)
{
    kv_t *kv = (kv_t *)malloc(sizeof(kv_t) * (size_t)k);
    for (int j = 0; j < k; j++) {
        int id = ids[j];
        double b = dl[id] / Td;
        double a = tl[id] / Tt;
        kv[j].v = b - a;
        kv[j].id = id;
    }
    qsort(kv, (size_t)k, sizeof(kv_t), cmp_key_desc);
    double Tg = 0.0, Dr = 0.0;
    psi_out[0] = 0.0; Tg_out[0] = 0.0; Dr_out[0] = 0.0;
    int jstar = 0; double best = 0.0;
    for (int j = 1; j <= k; j++) {
        int id = kv[j - 1].id;
        order_out[j - 1] = id;
        Tg += tgt[id]; Dr += drf[id];
        if (j == k) { Dr = 1.0; if (full_support) Tg = 1.0; }   /* both distributions are normalised */
        Tg_out[j] = Tg; Dr_out[j] = Dr;
        psi_out[j] = Tg - pow(Dr, (double)n);
        if (psi_out[j] < best) { best = psi_out[j]; jstar = j; }
    }
    free(kv);
    *alpha_star_out = 1.0 + best;
    return jstar;
}

/* ------------------------------------------------------------------ O4, O5
 * Outer residuals by the greedy polymatroid rule (Sec. 6.1, Thm "polymatroid",
 * Lemma "q-convex"): take V \ H* in INCREASING drf/tgt; then every
 * min_{T >= H_i} psi(T) lies among psi(H_i), ..., psi(H_1), so cumulative minima
 * of psi along the chain give
 *   p_v = tgt(v) + min_{T>=H_{i+1}} psi - min_{T>=H_i} psi,   r_v = tgt(v) - p_v.
 * Chain: V, then all zero-draft ids removed (psi = Tg_k - 1; each of them gets
 * p = 0, r = tgt), then the support positions k-1, k-2, ..., j* removed one by one
 * (psi_{k-s} after s removals).
 * Blocks: whenever the chain value is a new strict minimum the prefix Hall
 * inequality of the removed (lowest-ratio) tokens is tight, so tuples touching
 * them give them all their mass; the softmax system therefore splits there.
 * block_out[pos] = -1 on H*, else 0,1,... counted from the lowest ratio.
 * Returns the number of blocks.
 */
int gro_outer_residuals(const double *tgt_pos, const double *psi,
                        int k, int jstar, double *p_out, double *r_out, int *block_out)
{
    for (int j = 0; j < jstar; j++) { p_out[j] = tgt_pos[j]; r_out[j] = 0.0; block_out[j] = -1; }
    double m_prev = psi[k];                /* psi of the whole support = Tg_k - 1 */
    int blk = 0, open = 0;
    for (int s = 1; s <= k - jstar; s++) {
        int pos = k - s;
        double c = psi[k - s];
        int record = (c < m_prev);
        double m = record ? c : m_prev;
        r_out[pos] = m_prev - m;
        p_out[pos] = tgt_pos[pos] - r_out[pos];
        block_out[pos] = blk; open = 1;
        if (record) { blk++; open = 0; }
        m_prev = m;
    }
    return blk + open;
}

/* ------------------------------------------------------------------ gradients
 * Both convex programs (Thm "Outer Convex Solver", Thm "Inner Convex Solver")
 * have gradient  g_i(w) - rhs_i  with, for w_i = exp(alpha_i),
 *   inner:  g_i = sum_{omega in (H*)^n, i in set(omega)} drf^n(omega) w_i / (1 + sum_{j in set(omega)} w_j)
 *   outer block B with higher-ratio mass h:
 *           g_i = sum_{omega in (B u higher)^n, i in set(omega)} drf^n(omega) w_i / sum_{j in set(omega) n B} w_j
 * (Eqs. "defined-s-inner", "defined-s-outer" summed over the tuples).
 */

/* Route G1: grouped LogSumExp terms with inclusion-exclusion coefficients
 * (App. K): the weight of the term on exactly the set A is
 *   sum_{C subset A} (-1)^{|A|-|C|} (h + drf(C))^n      (h = 0 in the inner system).
 * Exponential in m; meant for m <= ~20. */
int gro_grad_g1(int m, const double *d, const double *w, int n, double h, int slack, double *g)
{
    if (m > 24) return GRO_BAD_ARG;
    for (int i = 0; i < m; i++) g[i] = 0.0;
    uint32_t full = (m == 32) ? 0xffffffffu : ((1u << m) - 1u);
    for (uint32_t A = 1; A <= full; A++) {
        int sz = __builtin_popcount(A);
        if (sz > n) continue;
        double coef = 0.0;
        /* all subsets C of A, including the empty one */
        uint32_t C = A;
        for (;;) {
            double dc = h;
            for (int j = 0; j < m; j++) if (C >> j & 1u) dc += d[j];
            int sgn = ((sz - __builtin_popcount(C)) & 1) ? -1 : 1;
            coef += sgn * pow(dc, (double)n);
            if (C == 0) break;
            C = (C - 1) & A;
        }
        double W = slack ? 1.0 : 0.0;
        for (int j = 0; j < m; j++) if (A >> j & 1u) W += w[j];
        for (int j = 0; j < m; j++) if (A >> j & 1u) g[j] += coef * w[j] / W;
    }
    return GRO_OK;
}

/* Route G2: the same sums through 1/W = int_0^inf exp(-tW) dt and the exponential
 * generating function of n i.i.d. draws.  With x_j(t) = exp(-t w_j),
 *   g_i = w_i int_0^inf x_i(t) [e^{-t}]  n! [lambda^n]{ e^{lambda h} (e^{lambda d_i}-1)
 *                      prod_{j != i} (1 + x_j(t)(e^{lambda d_j}-1)) } dt ,
 * the bracketed e^{-t} present only with the slack vertex (inner system).
 * The lambda-series are truncated at degree n; all coefficients are >= 0.
 * Quadrature: t = exp(s - exp(-s)) (double-exponential map of the half line),
 * trapezoid in s, step halved until the values settle.
 */
static void series_mul_factor(double *P, int n, double x, const double *E)
{
    /* P <- P * (1 + x * sum_{m>=1} E[m] lambda^m), truncated at degree n; in place, high to low */
    for (int c = n; c >= 1; c--) {
        double acc = P[c];
        for (int m = 1; m <= c; m++) acc += x * E[m] * P[c - m];
        P[c] = acc;
    }
}

static void g2_fixed_step(int m, const double *d, const double *w, int n, double h, int slack,
                          double step, double s_lo, double s_hi, double *g,
                          double *E, double *pre, double *suf, double *x)
{
    int n1 = n + 1;
    double nfact = 1.0;
    for (int c = 2; c <= n; c++) nfact *= c;
    for (int i = 0; i < m; i++) g[i] = 0.0;
    int Q = (int)floor((s_hi - s_lo) / step + 1e-9) + 1;
    for (int q = 0; q < Q; q++) {
        double s = s_lo + step * q;
        double t = exp(s - exp(-s));
        double wt = step * (1.0 + exp(-s)) * t;
        for (int j = 0; j < m; j++) x[j] = exp(-t * w[j]);
        /* pre[j] = e^{lambda h} prod_{l<j} factor_l ; suf[j] = prod_{l>=j} factor_l */
        double *P0 = pre;
        double hp = 1.0, fc = 1.0;
        for (int c = 0; c <= n; c++) { P0[c] = hp / fc; hp *= h; fc *= (c + 1); }
        for (int j = 0; j < m; j++) {
            double *Pn = pre + (size_t)(j + 1) * n1;
            memcpy(Pn, pre + (size_t)j * n1, sizeof(double) * n1);
            series_mul_factor(Pn, n, x[j], E + (size_t)j * n1);
        }
        double *Sm = suf + (size_t)m * n1;
        for (int c = 0; c <= n; c++) Sm[c] = (c == 0) ? 1.0 : 0.0;
        for (int j = m - 1; j >= 0; j--) {
            double *Sn = suf + (size_t)j * n1;
            memcpy(Sn, suf + (size_t)(j + 1) * n1, sizeof(double) * n1);
            series_mul_factor(Sn, n, x[j], E + (size_t)j * n1);
        }
        double damp = slack ? exp(-t) : 1.0;
        for (int i = 0; i < m; i++) {
            const double *A = pre + (size_t)i * n1, *B = suf + (size_t)(i + 1) * n1;
            const double *Ei = E + (size_t)i * n1;
            /* [lambda^n] A*B*Ei = sum_{a+b+e=n, e>=1} A[a] B[b] Ei[e] */
            double coef = 0.0;
            for (int e = 1; e <= n; e++) {
                double ab = 0.0;
                for (int a = 0; a <= n - e; a++) ab += A[a] * B[n - e - a];
                coef += ab * Ei[e];
            }
            g[i] += wt * damp * w[i] * x[i] * coef * nfact;
        }
    }
}

int gro_grad_g2(int m, const double *d, const double *w, int n, double h, int slack, double *g)
{
    if (m <= 0) return GRO_OK;
    int n1 = n + 1;
    double *E = (double *)malloc(sizeof(double) * (size_t)m * n1);
    double *pre = (double *)malloc(sizeof(double) * (size_t)(m + 1) * n1);
    double *suf = (double *)malloc(sizeof(double) * (size_t)(m + 1) * n1);
    double *x = (double *)malloc(sizeof(double) * (size_t)m);
    double *g2 = (double *)malloc(sizeof(double) * (size_t)m);
    for (int j = 0; j < m; j++) {
        double pw = 1.0, fc = 1.0;
        E[(size_t)j * n1] = 0.0;
        for (int c = 1; c <= n; c++) { pw *= d[j]; fc *= c; E[(size_t)j * n1 + c] = pw / fc; }
    }
    /* slowest decay rate of any integrand: (slack +) min_i w_i */
    double rmin = INFINITY;
    for (int j = 0; j < m; j++) if (w[j] < rmin) rmin = w[j];
    if (slack) rmin += 1.0;
    double s_lo = -5.0, s_hi = log(50.0 / rmin);
    if (s_hi < 1.0) s_hi = 1.0;
    double step = 0.25;
    g2_fixed_step(m, d, w, n, h, slack, step, s_lo, s_hi, g, E, pre, suf, x);
    int ok = 0;
    for (int lvl = 0; lvl < 8 && !ok; lvl++) {
        step *= 0.5;
        g2_fixed_step(m, d, w, n, h, slack, step, s_lo, s_hi, g2, E, pre, suf, x);
        ok = 1;
        for (int i = 0; i < m; i++) {
            if (fabs(g2[i] - g[i]) > 1e-15 + 2e-14 * fabs(g2[i])) ok = 0;
            g[i] = g2[i];
        }
    }
    free(E); free(pre); free(suf); free(x); free(g2);
    return ok ? GRO_OK : GRO_NOT_CONVERGED;
}

static int grad_route(int route, int m, const double *d, const double *w, int n, double h, int slack, double *g)
{
    return (route == 1) ? gro_grad_g1(m, d, w, n, h, slack, g) : gro_grad_g2(m, d, w, n, h, slack, g);
}

/* ------------------------------------------------------------------ O6, O7
 * Solve g(w) = rhs by iterative proportional fitting  w_i <- w_i rhs_i / g_i(w)
 * (row scaling of the softmax-parametrised flows with the tuple side eliminated);
 * the fixed point is the stationary point of Theta (slack=1) or of Phi restricted
 * to a block (slack=0).  Stops when ||g - rhs||_1 <= tol, which is the L1 norm
 * of the gradient of the convex function.  Outer blocks are scale free: after
 * every sweep the weights are renormalised to geometric mean 1.
 */
int gro_ipf(int route, int m, const double *d, const double *rhs, int n, double h, int slack,
            double tol, int max_iter, double *w, double *gnorm_out, int *iters_out)
{
    double *g = (double *)malloc(sizeof(double) * (size_t)(m > 0 ? m : 1));
    for (int i = 0; i < m; i++) w[i] = 1.0;
    int it = 0, status = GRO_NOT_CONVERGED;
    double gn = 0.0;
    if (m == 0) { status = GRO_OK; }
    for (; m > 0 && it <= max_iter; it++) {
        grad_route(route, m, d, w, n, h, slack, g);
        gn = 0.0;
        for (int i = 0; i < m; i++) gn += fabs(g[i] - rhs[i]);
        if (gn <= tol) { status = GRO_OK; break; }
        if (it == max_iter) break;
        for (int i = 0; i < m; i++) w[i] *= rhs[i] / g[i];
        if (!slack) {
            double sl = 0.0;
            for (int i = 0; i < m; i++) sl += log(w[i]);
            double sc = exp(-sl / m);
            for (int i = 0; i < m; i++) w[i] *= sc;
        }
    }
    free(g);
    if (gnorm_out) *gnorm_out = gn;
    if (iters_out) *iters_out = it;
    return status;
}

/* Damped Newton on the same equations, in alpha = log w.  The Jacobian of g is taken
 * by central differences of the gradient routine (the Hessian of the convex function);
 * it only steers the iteration: the stopping test is the L1 gradient norm evaluated by
 * the gradient routine itself, and the stationary point is unique (strict convexity
 * inside a block), so any iteration that passes the test returns the same weights.
 * A few proportional-fitting sweeps come first; a Newton step that does not reduce the
 * norm after backtracking is replaced by one more such sweep.
 */
static int lin_solve(int m, double *A, double *b)
{
    for (int c = 0; c < m; c++) {
        int piv = c; double best = fabs(A[(size_t)c * m + c]);
        for (int r2 = c + 1; r2 < m; r2++) if (fabs(A[(size_t)r2 * m + c]) > best) { best = fabs(A[(size_t)r2 * m + c]); piv = r2; }
        if (best == 0.0) return -1;
        if (piv != c) {
            for (int q = 0; q < m; q++) { double t = A[(size_t)c * m + q]; A[(size_t)c * m + q] = A[(size_t)piv * m + q]; A[(size_t)piv * m + q] = t; }
            double t = b[c]; b[c] = b[piv]; b[piv] = t;
        }
        for (int r2 = c + 1; r2 < m; r2++) {
            double f = A[(size_t)r2 * m + c] / A[(size_t)c * m + c];
            if (f == 0.0) continue;
            for (int q = c; q < m; q++) A[(size_t)r2 * m + q] -= f * A[(size_t)c * m + q];
            b[r2] -= f * b[c];
        }
    }
    for (int c = m - 1; c >= 0; c--) {
        double acc = b[c];
        for (int q = c + 1; q < m; q++) acc -= A[(size_t)c * m + q] * b[q];
        b[c] = acc / A[(size_t)c * m + c];
    }
    return 0;
}

static double resid_l1(int route, int m, const double *d, const double *rhs, int n, double h, int slack,
                       const double *alpha, double *w, double *g)
{
    for (int i = 0; i < m; i++) w[i] = exp(alpha[i]);
    grad_route(route, m, d, w, n, h, slack, g);
    double gn = 0.0;
    for (int i = 0; i < m; i++) gn += fabs(g[i] - rhs[i]);
    return gn;
}

int gro_newton(int route, int m, const double *d, const double *rhs, int n, double h, int slack,
               double tol, int max_iter, double *w, double *gnorm_out, int *iters_out)
{
    if (m == 0) { if (gnorm_out) *gnorm_out = 0.0; if (iters_out) *iters_out = 0; return GRO_OK; }
    const int ipf_sweeps = 10;
    const double delta = 1e-4;
    size_t mm = (size_t)m;
    double *alpha = (double *)calloc(mm, sizeof(double));
    double *trial = (double *)malloc(sizeof(double) * mm);
    double *g = (double *)malloc(sizeof(double) * mm);
    double *gp = (double *)malloc(sizeof(double) * mm);
    double *gm = (double *)malloc(sizeof(double) * mm);
    double *step = (double *)malloc(sizeof(double) * mm);
    double *J = (double *)malloc(sizeof(double) * mm * mm);
    int status = GRO_NOT_CONVERGED, it = 0;
    double gn = resid_l1(route, m, d, rhs, n, h, slack, alpha, w, g);
    for (; it < max_iter; it++) {
        if (gn <= tol) { status = GRO_OK; break; }
        int did_newton = 0;
        if (it >= ipf_sweeps) {
            for (int j = 0; j < m; j++) {
                memcpy(trial, alpha, sizeof(double) * mm);
                trial[j] = alpha[j] + delta; resid_l1(route, m, d, rhs, n, h, slack, trial, w, gp);
                trial[j] = alpha[j] - delta; resid_l1(route, m, d, rhs, n, h, slack, trial, w, gm);
                for (int i = 0; i < m; i++) J[(size_t)i * mm + j] = (gp[i] - gm[i]) / (2.0 * delta);
            }
            if (!slack) for (size_t q = 0; q < mm * mm; q++) J[q] += 1.0 / m;   /* pins the free common shift */
            resid_l1(route, m, d, rhs, n, h, slack, alpha, w, g);
            for (int i = 0; i < m; i++) step[i] = -(g[i] - rhs[i]);
            if (lin_solve(m, J, step) == 0) {
                double lam = 1.0;
                while (lam > 1e-4) {
                    for (int i = 0; i < m; i++) trial[i] = alpha[i] + lam * step[i];
                    double gt = resid_l1(route, m, d, rhs, n, h, slack, trial, w, gp);
                    if (gt < (1.0 - 1e-4 * lam) * gn) { memcpy(alpha, trial, sizeof(double) * mm); gn = gt; did_newton = 1; break; }
                    lam *= 0.5;
                }
            }
        }
        if (!did_newton) {
            resid_l1(route, m, d, rhs, n, h, slack, alpha, w, g);
            for (int i = 0; i < m; i++) alpha[i] += log(rhs[i] / g[i]);
        }
        if (!slack) {
            double mean = 0.0;
            for (int i = 0; i < m; i++) mean += alpha[i];
            mean /= m;
            for (int i = 0; i < m; i++) alpha[i] -= mean;
        }
        if (!did_newton || !slack) gn = resid_l1(route, m, d, rhs, n, h, slack, alpha, w, g);
    }
    if (gn <= tol) status = GRO_OK;
    for (int i = 0; i < m; i++) w[i] = exp(alpha[i]);
    if (gnorm_out) *gnorm_out = gn;
    if (iters_out) *iters_out = it;
    free(alpha); free(trial); free(g); free(gp); free(gm); free(step); free(J);
    return status;
}

/* ------------------------------------------------------------------ truncation sets
 * Sec. 6.2 (tunable errors), Sec. 6.3 and Algorithm 1: the convex functions are minimised over a truncation
 * set T only, chosen minimal with
 *   inner:  T subset of H*,      gamma_T   = drf(H*)^n - drf(T)^n      <= tau,
 *   outer:  T subset of V \ H*,  epsilon_T = 1 - (drf(H*) + drf(T))^n  <= tau.
 * Fewest tokens for a given draft mass: tokens are taken in decreasing drf (equal drf: smaller id first) until
 * the bound holds; zero-draft ids never enter.  tau <= 0 keeps every support token (both errors zero).
 * Arrays are in ratio order (positions 0..jstar-1 = H*); in_T[pos] = 1 / 0.
 */
typedef struct { double d; int id; int pos; } tr_t;
static int cmp_tr(const void *a, const void *b)
{
    const tr_t *x = (const tr_t *)a, *y = (const tr_t *)b;
    if (x->d > y->d) return -1;
    if (x->d < y->d) return 1;
    return (x->id < y->id) ? -1 : (x->id > y->id);
}
int gro_truncation_sets(int k, int jstar, const int *order, const double *drf_pos, int n, double tau, int *in_T,
                        double *gamma_out, double *eps_out)
{
    double D = 0.0;
    for (int j = 0; j < jstar; j++) D += drf_pos[j];
    double Dn = pow(D, (double)n);
    if (!(tau > 0.0)) {
        for (int j = 0; j < k; j++) in_T[j] = 1;
        if (gamma_out) *gamma_out = 0.0;
        if (eps_out) *eps_out = 0.0;
        return GRO_OK;
    }
    tr_t *t = (tr_t *)malloc(sizeof(tr_t) * (size_t)(k > 0 ? k : 1));
    for (int j = 0; j < k; j++) in_T[j] = 0;
    /* inner */
    for (int j = 0; j < jstar; j++) { t[j].d = drf_pos[j]; t[j].id = order[j]; t[j].pos = j; }
    qsort(t, (size_t)jstar, sizeof(tr_t), cmp_tr);
    double c = 0.0, gam = Dn;
    for (int j = 0; j < jstar && gam > tau; j++) {
        c += t[j].d; in_T[t[j].pos] = 1;
        gam = Dn - pow(c, (double)n);
    }
    if (gamma_out) *gamma_out = gam > 0.0 ? gam : 0.0;
    /* outer */
    int mo = k - jstar;
    for (int j = 0; j < mo; j++) { t[j].d = drf_pos[jstar + j]; t[j].id = order[jstar + j]; t[j].pos = jstar + j; }
    qsort(t, (size_t)mo, sizeof(tr_t), cmp_tr);
    c = D;
    double eps = 1.0 - Dn;
    for (int j = 0; j < mo && eps > tau; j++) {
        c += t[j].d; in_T[t[j].pos] = 1;
        eps = 1.0 - pow(c, (double)n);
    }
    if (eps_out) *eps_out = eps > 0.0 ? eps : 0.0;
    free(t);
    return GRO_OK;
}

/* ------------------------------------------------------------------ whole solve
 * Steps 1-3 of the method for one decode position.  All per-support arrays are in
 * ratio order (position 0 = largest drf/tgt) and have k entries (psi: k+1).
 * method: 1 = proportional fitting alone, 2 = damped Newton (default).
 * tau > 0 (Algorithm 1): each system is solved on its truncation set alone, to gradient norm 5 tau (`tol` is
 * then not used); the weights of the tokens outside the sets are 0 (the guarantees of Thms "Inner / Outer
 * Convex Solver" hold for any value there).  For an outer block the tuples counted are those inside
 * (H* u T)^n, so its higher-ratio mass is drf(H*) plus the T-part of the higher outer blocks.
 */
int gro_solve(const double *tl, const double *dl, int V, int n, int topk, double Tt, double Td,
              int route, int method, double tol, int max_iter, double tau,
              double *tgt_full, double *drf_full,
              int *k_out, int *order, double *tgt_pos, double *drf_pos, double *psi,
              int *jstar_out, double *alpha_star_out, double *p, double *r, int *block, int *nblocks_out,
              double *w, double *gnorm_out, int *iters_out)
{
    if (V <= 0 || n <= 0) return GRO_BAD_ARG;
    int *ids = (int *)malloc(sizeof(int) * (size_t)V);
    int k = gro_distributions(tl, dl, V, topk, Tt, Td, tgt_full, drf_full, ids, NULL);
    if (k < 0) { free(ids); return k; }
    double *Tg = (double *)malloc(sizeof(double) * (size_t)(k + 1));
    double *Dr = (double *)malloc(sizeof(double) * (size_t)(k + 1));
    int jstar = gro_subset_selection(tl, dl, tgt_full, drf_full, ids, k, n, Tt, Td, k == V, order, psi, Tg, Dr, alpha_star_out);
    for (int j = 0; j < k; j++) { tgt_pos[j] = tgt_full[order[j]]; drf_pos[j] = drf_full[order[j]]; }
    int nb = gro_outer_residuals(tgt_pos, psi, k, jstar, p, r, block);
    *k_out = k; *jstar_out = jstar; *nblocks_out = nb;

    int status = GRO_OK, iters = 0; double gnorm = 0.0;
    if (tau > 0.0) {
        /* truncated variant: gather each system's T-part, solve it to 5 tau, scatter the weights back */
        int *in_T = (int *)malloc(sizeof(int) * (size_t)(k > 0 ? k : 1));
        int *map = (int *)malloc(sizeof(int) * (size_t)(k > 0 ? k : 1));
        double *dT = (double *)malloc(sizeof(double) * (size_t)(3 * k + 3));
        double *rT = dT + k + 1, *wT = rT + k + 1;
        gro_truncation_sets(k, jstar, order, drf_pos, n, tau, in_T, NULL, NULL);
        for (int j = 0; j < k; j++) w[j] = 0.0;
        double stop = 5.0 * tau;
        int m = 0;
        for (int j = 0; j < jstar; j++) if (in_T[j]) { dT[m] = drf_pos[j]; rT[m] = tgt_pos[j]; map[m] = j; m++; }
        if (m > 0) {
            double gn = 0.0; int it = 0;
            int st = (method == 1) ? gro_ipf(route, m, dT, rT, n, 0.0, 1, stop, max_iter, wT, &gn, &it)
                                   : gro_newton(route, m, dT, rT, n, 0.0, 1, stop, max_iter, wT, &gn, &it);
            if (st != GRO_OK) status = GRO_NOT_CONVERGED;
            gnorm += gn; iters += it;
            for (int q = 0; q < m; q++) w[map[q]] = wT[q];
        }
        double DH = 0.0;
        for (int j = 0; j < jstar; j++) DH += drf_pos[j];
        for (int b = nb - 1; b >= 0; b--) {         /* from the highest ratio down, the T-mass above accumulates */
            int lo = -1, hi = -1;
            for (int j = jstar; j < k; j++) if (block[j] == b) { if (lo < 0) lo = j; hi = j; }
            if (lo < 0) continue;
            double hT = DH;
            for (int j = jstar; j < lo; j++) if (in_T[j]) hT += drf_pos[j];
            m = 0;
            for (int j = lo; j <= hi; j++) if (in_T[j]) { dT[m] = drf_pos[j]; rT[m] = p[j]; map[m] = j; m++; }
            if (m == 1) w[map[0]] = 1.0;
            if (m >= 2) {
                double gn = 0.0; int it = 0;
                int st = (method == 1) ? gro_ipf(route, m, dT, rT, n, hT, 0, stop, max_iter, wT, &gn, &it)
                                       : gro_newton(route, m, dT, rT, n, hT, 0, stop, max_iter, wT, &gn, &it);
                if (st != GRO_OK) status = GRO_NOT_CONVERGED;
                gnorm += gn; iters += it;
                for (int q = 0; q < m; q++) w[map[q]] = wT[q];
            }
        }
        free(in_T); free(map); free(dT);
        if (gnorm_out) *gnorm_out = gnorm;
        if (iters_out) *iters_out = iters;
        free(ids); free(Tg); free(Dr);
        return status;
    }
    /* inner system on H* (positions 0..jstar-1), rhs = tgt */
    {
        double gn = 0.0; int it = 0;
        int st = (method == 1) ? gro_ipf(route, jstar, drf_pos, tgt_pos, n, 0.0, 1, tol, max_iter, w, &gn, &it)
                               : gro_newton(route, jstar, drf_pos, tgt_pos, n, 0.0, 1, tol, max_iter, w, &gn, &it);
        if (st != GRO_OK) status = GRO_NOT_CONVERGED;
        gnorm += gn; iters += it;
    }
    /* outer blocks: contiguous position ranges, higher-ratio mass h = Dr[lo] */
    for (int b = 0; b < nb; b++) {
        int lo = -1, hi = -1;
        for (int j = jstar; j < k; j++) if (block[j] == b) { if (lo < 0) lo = j; hi = j; }
        if (lo < 0) continue;
        int m = hi - lo + 1;
        if (m == 1) { w[lo] = 1.0; continue; }
        double gn = 0.0; int it = 0;
        int st = (method == 1) ? gro_ipf(route, m, drf_pos + lo, p + lo, n, Dr[lo], 0, tol, max_iter, w + lo, &gn, &it)
                               : gro_newton(route, m, drf_pos + lo, p + lo, n, Dr[lo], 0, tol, max_iter, w + lo, &gn, &it);
        if (st != GRO_OK) status = GRO_NOT_CONVERGED;
        gnorm += gn; iters += it;
    }
    if (gnorm_out) *gnorm_out = gnorm;
    if (iters_out) *iters_out = iters;
    free(ids); free(Tg); free(Dr);
    return status;
}

/* ------------------------------------------------------------------ O8
 * One slice of the transport (Eq. "cases", Eq. "approx-c", "normalized" in
 * Algorithm 1).  U = distinct drafted tokens in order of first occurrence.
 *   all of U in H*:  pi(i) = w_i / (1 + sum_U w),  rho = 1 / (1 + sum_U w) goes to
 *                    the resample distribution r / (1 - alpha*);
 *   otherwise:       B = lowest-ratio block met by U; pi(i) = w_i / sum_{U n B} w on
 *                    U n B, 0 on the rest of U, rho = 0.  (Truncated variant: when every
 *                    token of U n B carries weight 0 they share the tuple equally.)
 * U_out / pi_out have up to n entries; returns |U| or a negative error.
 */
int gro_slice(int k, int n, int jstar, const int *order, const int *block, const double *w,
              const int *omega, int *U_out, double *pi_out, double *rho_out)
{
    int *pos = (int *)malloc(sizeof(int) * (size_t)n);
    int nu = 0;
    for (int s = 0; s < n; s++) {
        int found = -1;
        for (int j = 0; j < k; j++) if (order[j] == omega[s]) { found = j; break; }
        if (found < 0) { free(pos); return GRO_DRAFT_OUT_OF_SUPPORT; }
        int dup = 0;
        for (int u = 0; u < nu; u++) if (pos[u] == found) dup = 1;
        if (!dup) { pos[nu] = found; U_out[nu] = omega[s]; nu++; }
    }
    int maxpos = -1;
    for (int u = 0; u < nu; u++) if (pos[u] > maxpos) maxpos = pos[u];
    if (maxpos < jstar) {
        double W = 1.0;
        for (int u = 0; u < nu; u++) W += w[pos[u]];
        for (int u = 0; u < nu; u++) pi_out[u] = w[pos[u]] / W;
        *rho_out = 1.0 / W;
    } else {
        int b = block[maxpos];
        double W = 0.0;
        int cnt = 0;
        for (int u = 0; u < nu; u++) if (block[pos[u]] == b) { W += w[pos[u]]; cnt++; }
        for (int u = 0; u < nu; u++)
            pi_out[u] = (block[pos[u]] == b) ? (W > 0.0 ? w[pos[u]] / W : 1.0 / cnt) : 0.0;
        *rho_out = 0.0;
    }
    free(pos);
    return nu;
}

/* ------------------------------------------------------------------ O9
 * Draw (App. A, steps 3-4): segments are U's tokens in first-occurrence order,
 * then the resample segment; the emitted segment is the first whose cumulative
 * probability exceeds u0.  In the resample segment the token is the first id t
 * (ascending) whose cumulative residual exceeds u1 times the total residual.
 * r_full[i] = tgt_i off the support, the outer residual on outer support ids, 0 on H*.
 */
int gro_draw(int nu, const int *U, const double *pi, double rho, const double *r_full, int V,
             double u0, double u1, int *token_out, int *accepted_out)
{
    double c = 0.0;
    int last_pos = -1;
    for (int u = 0; u < nu; u++) {
        c += pi[u];
        if (pi[u] > 0.0) last_pos = u;
        if (c > u0) { *token_out = U[u]; *accepted_out = 1; return GRO_OK; }
    }
    if (!(rho > 0.0)) { *token_out = U[last_pos]; *accepted_out = 1; return GRO_OK; }
    double tot = 0.0;
    for (int i = 0; i < V; i++) tot += r_full[i];
    double thr = u1 * tot, acc = 0.0;
    int last = -1;
    for (int i = 0; i < V; i++) {
        acc += r_full[i];
        if (r_full[i] > 0.0) last = i;
        if (acc > thr) { *token_out = i; *accepted_out = 0; return GRO_OK; }
    }
    *token_out = last; *accepted_out = 0;
    return GRO_OK;
}

/* ------------------------------------------------------------------ batch driver
 * Solve + slice + draw for a batch (instances are independent; OpenMP over them).
 * Logits are row-major [batch, V] doubles (exact upcasts of the fp32/bf16 inputs).
 * Per-instance outputs: alpha_star, token, accepted, status, and -- when the
 * pointers are not NULL -- the slice (U padded with -1, pi padded with 0, rho).
 */
int gro_solve_verify_batch(const double *tl, const double *dl, int batch, int V, int n, int topk,
                           double Tt, double Td, int route, int method, double tol, int max_iter, double tau,
                           const int *draft_tokens, const float *uniforms,
                           double *alpha_star, int *token, int *accepted, int *status,
                           int *U_out, double *pi_out, double *rho_out, double *gnorm_out, int *iters_out,
                           int *jstar_out,
                           int kcap, int *k_out, int *nblocks_out, int *order_out, int *block_out,
                           double *w_out, double *r_out, double *p_out, double *psi_out)
{
    /* the last group of outputs is optional (NULL skips): the whole solution of every instance, per-support arrays
     * with kcap entries per instance in ratio order (psi: kcap + 1), unused entries -1 / 0 */
    int k = (topk <= 0 || topk >= V) ? V : topk;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < batch; b++) {
        const double *tlb = tl + (size_t)b * V, *dlb = dl + (size_t)b * V;
        double *tgt = (double *)malloc(sizeof(double) * (size_t)V);
        double *drf = (double *)malloc(sizeof(double) * (size_t)V);
        int *order = (int *)malloc(sizeof(int) * (size_t)k);
        int *block = (int *)malloc(sizeof(int) * (size_t)k);
        double *buf = (double *)malloc(sizeof(double) * (size_t)(6 * k + 1));
        double *tgt_pos = buf, *drf_pos = buf + k, *psi = buf + 2 * k, *p = buf + 3 * k + 1,
               *r = buf + 4 * k + 1, *w = buf + 5 * k + 1;
        int kk = 0, jstar = 0, nb = 0, iters = 0; double gn = 0.0, as = 0.0;
        int st = gro_solve(tlb, dlb, V, n, topk, Tt, Td, route, method, tol, max_iter, tau, tgt, drf, &kk, order,
                           tgt_pos, drf_pos, psi, &jstar, &as, p, r, block, &nb, w, &gn, &iters);
        alpha_star[b] = as;
        if (gnorm_out) gnorm_out[b] = gn;
        if (iters_out) iters_out[b] = iters;
        if (jstar_out) jstar_out[b] = jstar;
        if (k_out) k_out[b] = kk;
        if (nblocks_out) nblocks_out[b] = nb;
        for (int j = 0; j < kcap; j++) {
            size_t o = (size_t)b * kcap + j;
            int in = j < kk;
            if (order_out) order_out[o] = in ? order[j] : -1;
            if (block_out) block_out[o] = in ? block[j] : -2;
            if (w_out) w_out[o] = in ? w[j] : 0.0;
            if (r_out) r_out[o] = in ? r[j] : 0.0;
            if (p_out) p_out[o] = in ? p[j] : 0.0;
        }
        if (psi_out) for (int j = 0; j <= kcap; j++) psi_out[(size_t)b * (kcap + 1) + j] = j <= kk ? psi[j] : 0.0;
        int *U = (int *)malloc(sizeof(int) * (size_t)n);
        double *pi = (double *)malloc(sizeof(double) * (size_t)n);
        double rho = 0.0;
        int nu = gro_slice(kk, n, jstar, order, block, w, draft_tokens + (size_t)b * n, U, pi, &rho);
        if (nu < 0) {
            status[b] = nu; token[b] = -1; accepted[b] = 0;
        } else {
            /* dense residual vector: tgt off the support, outer residual on it */
            for (int j = 0; j < kk; j++) tgt[order[j]] = r[j];
            int tk = -1, ac = 0;
            gro_draw(nu, U, pi, rho, tgt, V, (double)uniforms[2 * b], (double)uniforms[2 * b + 1], &tk, &ac);
            token[b] = tk; accepted[b] = ac; status[b] = st;
        }
        if (U_out) for (int s = 0; s < n; s++) U_out[(size_t)b * n + s] = (nu > 0 && s < nu) ? U[s] : -1;
        if (pi_out) for (int s = 0; s < n; s++) pi_out[(size_t)b * n + s] = (nu > 0 && s < nu) ? pi[s] : 0.0;
        if (rho_out) rho_out[b] = (nu > 0) ? rho : 0.0;
        free(U); free(pi); free(tgt); free(drf); free(order); free(block); free(buf);
    }
    return GRO_OK;
}

/* ------------------------------------------------------------------ certificate
 * The structure of every instance (distributions, ratio order, H*, residuals, blocks: steps O1-O5, no convex
 * solve) and, for weights w_in given from outside (per-support arrays of kcap entries per instance in THIS
 * ratio order), the L1 norm of the gradient of the convex functions at those weights,
 *   || g_inner(w) - tgt ||_1 on H*  +  sum over outer blocks with >= 2 tokens of || g_block(w) - p ||_1
 * (Thm "Inner Convex Solver", Thm "Outer Convex Solver": the gradient of Theta / Phi is g - rhs), one gradient
 * evaluation per system by the integral route.  A small value certifies the weights: inside a system the
 * stationary point is unique.  Weights of positions outside every solved system are ignored.
 * lse_in (optional, NULL = none): a log-sum-exp of the target row per instance given from outside; cert2_out then
 * receives the same norm with the target normalised by THAT value (tgt_i = exp(tl_i / Tt - lse_in)), which separates
 * the error of the weights from the error of the normalisation they were solved for.  The structure always comes
 * from the oracle's own distributions.
 */
int gro_certify_batch(const double *tl, const double *dl, int batch, int V, int n, int topk, double Tt, double Td,
                      const double *w_in, int kcap, const double *lse_in, double *cert2_out, double *lse_out,
                      int *k_out, int *jstar_out, int *nblocks_out, double *alpha_star_out,
                      int *order_out, int *block_out, double *r_out, double *p_out, double *psi_out,
                      double *cert_out)
{
    int k = (topk <= 0 || topk >= V) ? V : topk;
    if (k > kcap) return GRO_BAD_ARG;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < batch; b++) {
        const double *tlb = tl + (size_t)b * V, *dlb = dl + (size_t)b * V;
        double *tgt = (double *)malloc(sizeof(double) * (size_t)V);
        double *drf = (double *)malloc(sizeof(double) * (size_t)V);
        int *ids = (int *)malloc(sizeof(int) * (size_t)V);
        int *order = (int *)malloc(sizeof(int) * (size_t)k);
        int *block = (int *)malloc(sizeof(int) * (size_t)k);
        double *buf = (double *)malloc(sizeof(double) * (size_t)(8 * k + 3));
        double *tgt_pos = buf, *drf_pos = buf + k, *psi = buf + 2 * k, *p = buf + 3 * k + 1, *r = buf + 4 * k + 1,
               *Tg = buf + 5 * k + 1, *Dr = buf + 6 * k + 2, *g = buf + 7 * k + 3;
        double lse_own = 0.0;
        int kk = gro_distributions(tlb, dlb, V, topk, Tt, Td, tgt, drf, ids, &lse_own);
        if (lse_out) lse_out[b] = lse_own;
        double as = 0.0;
        int jstar = gro_subset_selection(tlb, dlb, tgt, drf, ids, kk, n, Tt, Td, kk == V, order, psi, Tg, Dr, &as);
        for (int j = 0; j < kk; j++) { tgt_pos[j] = tgt[order[j]]; drf_pos[j] = drf[order[j]]; }
        int nb = gro_outer_residuals(tgt_pos, psi, kk, jstar, p, r, block);
        const double *w = w_in + (size_t)b * kcap;
        /* right-hand sides under the outside normalisation: targets rescaled, the chain psi = Tg - Dr^n and the
         * residuals recomputed from them (block boundaries kept) */
        double scale2 = lse_in ? exp(lse_own - lse_in[b]) : 1.0;
        double *tgt2 = (double *)malloc(sizeof(double) * (size_t)(3 * kk + 2));
        double *psi2 = tgt2 + kk, *p2 = psi2 + kk + 1;
        double *r2 = (double *)malloc(sizeof(double) * (size_t)(kk + 1));
        int *block2 = (int *)malloc(sizeof(int) * (size_t)(kk + 1));
        for (int j = 0; j < kk; j++) tgt2[j] = tgt_pos[j] * scale2;
        for (int j = 0; j <= kk; j++) psi2[j] = Tg[j] * scale2 - (Tg[j] - psi[j]);
        gro_outer_residuals(tgt2, psi2, kk, jstar, p2, r2, block2);
        double cert = 0.0, cert2 = 0.0;
        if (jstar > 0) {
            gro_grad_g2(jstar, drf_pos, w, n, 0.0, 1, g);
            for (int i = 0; i < jstar; i++) { cert += fabs(g[i] - tgt_pos[i]); cert2 += fabs(g[i] - tgt_pos[i] * scale2); }
        }
        for (int bk = 0; bk < nb; bk++) {
            int lo = -1, hi = -1;
            for (int j = jstar; j < kk; j++) if (block[j] == bk) { if (lo < 0) lo = j; hi = j; }
            if (lo < 0 || hi == lo) continue;
            int m = hi - lo + 1;
            gro_grad_g2(m, drf_pos + lo, w + lo, n, Dr[lo], 0, g);
            for (int i = 0; i < m; i++) { cert += fabs(g[i] - p[lo + i]); cert2 += fabs(g[i] - p2[lo + i]); }
        }
        if (cert2_out) cert2_out[b] = cert2;
        free(tgt2); free(r2); free(block2);
        k_out[b] = kk; jstar_out[b] = jstar; nblocks_out[b] = nb; alpha_star_out[b] = as; cert_out[b] = cert;
        for (int j = 0; j < kcap; j++) {
            size_t o = (size_t)b * kcap + j;
            int in = j < kk;
            order_out[o] = in ? order[j] : -1;
            block_out[o] = in ? block[j] : -2;
            r_out[o] = in ? r[j] : 0.0;
            p_out[o] = in ? p[j] : 0.0;
        }
        for (int j = 0; j <= kcap; j++) psi_out[(size_t)b * (kcap + 1) + j] = j <= kk ? psi[j] : 0.0;
        free(tgt); free(drf); free(ids); free(order); free(block); free(buf);
    }
    return GRO_OK;
}

/* ------------------------------------------------------------------ marginals of a rule
 * For ANY weights (zeros allowed, as the truncated variant leaves them) the rule of gro_slice defines a coupling;
 * this returns what Lemma "Approximation Guarantee" bounds: the L1 distance of its emitted-token marginal from the
 * target and its acceptance (= sum of the flows p'_i the tokens receive from the tuples that contain them).
 * Flows by the integral route: the inner system on all of H* with the given weights; per outer block the
 * tokens of positive weight (the block's zero-weight tokens take nothing from tuples that contain one of those,
 * so their mass joins the higher-ratio mass), and the zero-weight tokens among themselves with equal weights.
 * Emitted marginal (Eq. "approx-c"): p'_i on H*; p'_i + r_i rho / R on outer support tokens; tgt_i rho / R off the
 * support, with rho = drf(H*)^n - sum_{H*} p'_j the mass left to the resample segment and R = 1 - alpha*.
 * Arrays in ratio order, k entries; Dr = prefix sums of drf (k + 1 entries).
 */
int gro_rule_deviation(int k, int n, int jstar, int nblocks, const int *block, const double *tgt_pos,
                       const double *drf_pos, const double *r, const double *w, double alpha_star,
                       double *l1_out, double *accept_out, double *flow_out)
{
    double *flow = (double *)calloc((size_t)(k > 0 ? k : 1), sizeof(double));
    double *dd = (double *)malloc(sizeof(double) * (size_t)(3 * k + 3));
    double *ww = dd + k + 1, *gg = ww + k + 1;
    int *map = (int *)malloc(sizeof(int) * (size_t)(k > 0 ? k : 1));
    double DH = 0.0, tsup = 0.0;
    for (int j = 0; j < jstar; j++) DH += drf_pos[j];
    for (int j = 0; j < k; j++) tsup += tgt_pos[j];
    if (jstar > 0) {
        gro_grad_g2(jstar, drf_pos, w, n, 0.0, 1, gg);
        for (int j = 0; j < jstar; j++) flow[j] = w[j] > 0.0 ? gg[j] : 0.0;
    }
    double above = DH;                 /* draft mass of everything of higher ratio than the current block */
    for (int b = nblocks - 1; b >= 0; b--) {
        int lo = -1, hi = -1;
        for (int j = jstar; j < k; j++) if (block[j] == b) { if (lo < 0) lo = j; hi = j; }
        if (lo < 0) continue;
        double dz = 0.0;
        int mp = 0, mz = 0;
        for (int j = lo; j <= hi; j++) if (!(w[j] > 0.0)) dz += drf_pos[j];
        for (int j = lo; j <= hi; j++) if (w[j] > 0.0) { dd[mp] = drf_pos[j]; ww[mp] = w[j]; map[mp] = j; mp++; }
        if (mp > 0) {
            gro_grad_g2(mp, dd, ww, n, above + dz, 0, gg);
            for (int q = 0; q < mp; q++) flow[map[q]] = gg[q];
        }
        for (int j = lo; j <= hi; j++) if (!(w[j] > 0.0)) { dd[mz] = drf_pos[j]; ww[mz] = 1.0; map[mz] = j; mz++; }
        if (mz > 0) {
            gro_grad_g2(mz, dd, ww, n, above, 0, gg);
            for (int q = 0; q < mz; q++) flow[map[q]] = gg[q];
        }
        for (int j = lo; j <= hi; j++) above += drf_pos[j];
    }
    double acc = 0.0, inner_flow = 0.0;
    for (int j = 0; j < k; j++) acc += flow[j];
    for (int j = 0; j < jstar; j++) inner_flow += flow[j];
    double rho = pow(DH, (double)n) - inner_flow;
    double R = 1.0 - alpha_star;
    double share = R > 0.0 ? rho / R : 0.0;
    double l1 = 0.0;
    for (int j = 0; j < jstar; j++) l1 += fabs(flow[j] - tgt_pos[j]);
    for (int j = jstar; j < k; j++) l1 += fabs(flow[j] + r[j] * share - tgt_pos[j]);
    l1 += (1.0 - tsup) * fabs(share - 1.0);
    if (l1_out) *l1_out = l1;
    if (accept_out) *accept_out = acc;
    if (flow_out) for (int j = 0; j < k; j++) flow_out[j] = flow[j];
    free(flow); free(dd); free(map);
    return GRO_OK;
}

/* ------------------------------------------------------------------ draw sweep
 * Many draws from one solved rule per instance (App. A steps 3-4 through gro_slice / gro_draw): for R pairs of
 * uniforms per instance the emitted token and accepted flag, and how far the deciding uniform is from the nearest
 * boundary of the CDF it was compared with (the parity tests excuse a differing token only within 1e-6 of one).
 * The rule is given as per-support arrays of kcap entries per instance in ratio order (as gro_solve_verify_batch
 * returns them); uniforms are [batch, R, 2].
 */
int gro_draw_sweep_batch(const double *tl, const double *dl, int batch, int V, int n, int topk, double Tt, double Td,
                         int kcap, const int *k_in, const int *jstar_in, const int *order_in, const int *block_in,
                         const double *w_in, const double *r_in, const int *draft_tokens, const float *uniforms, int R,
                         int *token_out, int *accepted_out, double *margin_out)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < batch; b++) {
        const double *tlb = tl + (size_t)b * V, *dlb = dl + (size_t)b * V;
        double *rfull = (double *)malloc(sizeof(double) * (size_t)V);
        double *drf = (double *)malloc(sizeof(double) * (size_t)V);
        double *cum = (double *)malloc(sizeof(double) * (size_t)V);
        int *ids = (int *)malloc(sizeof(int) * (size_t)V);
        int *U = (int *)malloc(sizeof(int) * (size_t)n);
        double *pi = (double *)malloc(sizeof(double) * (size_t)n);
        gro_distributions(tlb, dlb, V, topk, Tt, Td, rfull, drf, ids, NULL);      /* rfull = tgt for now */
        const int kk = k_in[b];
        const int *order = order_in + (size_t)b * kcap, *block = block_in + (size_t)b * kcap;
        const double *w = w_in + (size_t)b * kcap, *r = r_in + (size_t)b * kcap;
        for (int j = 0; j < kk; j++) rfull[order[j]] = r[j];
        double tot = 0.0;
        for (int i = 0; i < V; i++) { tot += rfull[i]; }
        double acc = 0.0;
        for (int i = 0; i < V; i++) { acc += rfull[i]; cum[i] = acc; }            /* same summation order as gro_draw */
        double rho = 0.0;
        int nu = gro_slice(kk, n, jstar_in[b], order, block, w, draft_tokens + (size_t)b * n, U, pi, &rho);
        for (int q = 0; q < R; q++) {
            size_t o = (size_t)b * R + q;
            double u0 = (double)uniforms[2 * o], u1 = (double)uniforms[2 * o + 1];
            if (nu < 0) { token_out[o] = -1; accepted_out[o] = 0; margin_out[o] = 1.0; continue; }
            int tk = -1, ac = 0;
            gro_draw(nu, U, pi, rho, rfull, V, u0, u1, &tk, &ac);
            token_out[o] = tk; accepted_out[o] = ac;
            /* distance of u0 to the edges of the accepted segments */
            double mg = 1.0, c = 0.0;
            for (int u = 0; u < nu; u++) { c += pi[u]; if (fabs(c - u0) < mg) mg = fabs(c - u0); }
            if (!ac && tot > 0.0) {
                /* resample branch: distance of u1 to the CDF edges on either side of the emitted token */
                double thr = u1 * tot;
                double hi = cum[tk], lo = tk > 0 ? cum[tk - 1] : 0.0;
                double m1 = fabs(hi - thr) / tot, m0 = fabs(thr - lo) / tot;
                double mr = m1 < m0 ? m1 : m0;
                if (mr < mg) mg = mr;
            }
            margin_out[o] = mg;
        }
        free(rfull); free(drf); free(cum); free(ids); free(U); free(pi);
    }
    return GRO_OK;
}

int gro_num_threads(void)
{
    int nt = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        nt = omp_get_num_threads();
    }
#endif
    return nt;
}
