// Per-instance solve (one CTA per instance): subset selection, outer residuals,
// blocks, and the convex minimisation of the inner system and of every outer block.
//
// Gradient of the convex functions (Thm "Inner Convex Solver", Thm "Outer Convex
// Solver"): with w_i = exp(alpha_i) the i-th gradient entry is g_i(w) - rhs_i,
//   g_i = sum_{A containing i} Pr[set(omega) = A] w_i / (slack + sum_{j in A} w_j).
// The exponentially many terms are summed exactly through
//   1 / W = int_0^inf exp(-t W) dt   and   1 / W^2 = int_0^inf t exp(-t W) dt,
// and the exponential generating function of n i.i.d. draws:  with x_j = exp(-t w_j),
//   M(t) = n! [lambda^n] e^{lambda h} prod_j (1 + x_j (e^{lambda d_j} - 1)),
//   g_i = w_i int e^{-t slack} x_i dM/dx_i dt,
//   dg_i/dalpha_l = delta_il g_i - w_i w_l int t e^{-t slack} x_i x_l d2M/dx_i dx_l dt  (x_i for i = l),
//   dM/dx_i = n! [lambda^n] P h_i,   d2M/dx_i dx_l = n! [lambda^n] P h_i h_l,
//   P = e^{lambda h} prod_j f_j,  f_j = 1 + x_j e_j,  e_j = e^{lambda d_j} - 1,  h_j = e_j / f_j,
// all as power series in lambda truncated at degree n.  The t-integral is a
// trapezoid rule in s, t = exp(s - exp(-(s - s0))), which resolves every token's
// transition at t ~ 1/w_j on a logarithmic scale and closes the lower tail
// doubly exponentially.  Newton's method on alpha uses the exact Hessian above.
#include "gr_prep.cuh"
#include "gr_verify.cuh"

namespace gr {

constexpr int kSolveThreads = 256;
constexpr int kSolveWarps = kSolveThreads / 32;
constexpr int kGroups = 8;          // token groups whose partial products are combined per node
constexpr double kTEnd = 25.0;      // integrand below exp(-kTEnd) at the upper end
constexpr double kDrop = 1.0;       // the lower-tail compression starts this far below the fastest transition
constexpr double kTail = 3.0;       // and the grid extends this far below that
constexpr int kMaxNodes = 512;
constexpr double kAlphaClamp = 80.0;
constexpr double kStepClamp = 3.0;

struct SolveLayout {
    int KP, n, Qt;
    // offsets in doubles
    int d, tg, p, r, key, w, psi, Dr, alpha, alpha_prev, delta, g, g2, col, E, J, tq, cq, X, H, A, P, PP, PQ, PX, AX, gq, g2q, scal;
    int ints;      // offset in bytes of the int region
    int total_bytes;
    __host__ __device__ SolveLayout(int KP_, int n_, int Qt_) : KP(KP_), n(n_), Qt(Qt_) {
        int o = 0;
        d = o; o += KP; tg = o; o += KP; p = o; o += KP; r = o; o += KP; key = o; o += KP; w = o; o += KP;
        psi = o; o += KP + 4; Dr = o; o += KP + 4;
        alpha = o; o += KP; alpha_prev = o; o += KP; delta = o; o += KP; g = o; o += KP; g2 = o; o += KP;
        col = o; o += KP;
        E = o; o += KP * (n + 1);
        J = o; o += KP * (KP + 1) / 2;
        tq = o; o += Qt; cq = o; o += Qt;
        X = o; o += Qt * KP;
        H = o; o += Qt * (n + 1) * KP;
        A = o; o += Qt * (n + 1) * KP;
        P = o; o += Qt * (n + 1);
        PP = o; o += Qt * kGroups * (n + 1);
        PQ = o; o += Qt * kGroups * (n + 1);
        PX = o; o += Qt * 3 * (n + 1);
        AX = o; o += Qt * (n + 1);
        gq = o; o += Qt * KP; g2q = o; o += Qt * KP;
        scal = o; o += 32;
        ints = o * 8;
        total_bytes = ints + KP * 4 * 4 + 64;
    }
};

__host__ int solve_pick_tile(int KP, int n, int max_bytes) {
    int Qt = 32;
    while (Qt > 1 && SolveLayout(KP, n, Qt).total_bytes > max_bytes) Qt >>= 1;
    return Qt;
}
__host__ int solve_smem_bytes(int KP, int n, int Qt) { return SolveLayout(KP, n, Qt).total_bytes; }

struct Sm {
    GR_PTR(double) d, tg, p, r, key, w, psi, Dr, alpha, alpha_prev, delta, g, g2, col, E, J, tq, cq, X, H, A, P, PP, PQ, PX, AX,
        gq, g2q, scal;
    GR_PTR(int) id, blk, order, itmp;
    int KP, n, Qt;
};

__device__ inline int tri(int i, int l) { return i * (i + 1) / 2 + l; }   // l <= i

// scal[] slots
enum { S_WMAX = 0, S_WMIN, S_RNORM, S_RPREV, S_LAM, S_FAIL, S_DMAX, S_MEAN, S_SHI, S_S0, S_STEP, S_H, S_DA, S_DB,
       S_COARSE, S_PIVOT };
constexpr int S_ADD = S_MEAN;      // (slot reused: what was added to every Hessian entry)

// Evaluate g (and, if want_jac, the packed lower triangle of the Hessian) at sm.alpha[0..m).
// d = draft masses of the system's tokens, hmass = draft mass of everything of higher ratio
// (outer blocks), slack = 1 for the inner system.  Returns the number of quadrature nodes.
__device__ int eval_system(const Sm& sm, int m, GR_PTR(const double) d, double hmass, int slack, bool want_jac,
                           double qstep)
{
    const int tid = threadIdx.x;
    const int n = sm.n, n1 = sm.n + 1, KP = sm.KP, Qt = sm.Qt;
    GR_PTR(double) red = sm.scal + 16;
    // weights and their range
    double wj = 0.0;
    if (tid < m) { wj = exp(sm.alpha[tid]); sm.w[tid] = wj; sm.g[tid] = 0.0; sm.g2[tid] = 0.0; }
    double wmax = block_reduce_max(tid < m ? wj : 0.0, red);
    double wmin = -block_reduce_max(tid < m ? -wj : -1.0e300, red);
    if (want_jac)
        for (int e = tid; e < m * (m + 1) / 2; e += kSolveThreads) sm.J[e] = 0.0;
    const double rate = slack ? 1.0 + wmin : wmin;
    const double s_hi = log(kTEnd / rate);
    const double s0 = -log((slack ? 1.0 : 0.0) + wmax) - kDrop;
    int Q = (int)ceil((s_hi - (s0 - kTail)) / qstep) + 1;
    if (Q > kMaxNodes) Q = kMaxNodes;
    double nfact = 1.0;
    for (int c = 2; c <= n; c++) nfact *= (double)c;
    const int gsz = (m + kGroups - 1) / kGroups;
    // Dominant tokens (at most two; only for n > 16): the series division h = e / f would lose too many digits
    // for them, so their leave-one-out products are multiplied out instead (all coefficients positive).
    const int da = (int)sm.scal[S_DA], db = (int)sm.scal[S_DB];

    // e^{lambda h} = sum_c (h^c / c!) lambda^c, the same for every node
    if (tid <= n) {
        double v = 1.0;
        for (int a = 1; a <= tid; a++) v *= hmass / (double)a;
        sm.P[tid] = v;
    }
    for (int q0 = 0; q0 < Q; q0 += Qt) {
        const int qn = min(Qt, Q - q0);
        __syncthreads();
        if (tid < qn) {
            double s = s_hi - qstep * (double)(q0 + tid);
            double e = exp(-(s - s0));
            double t = exp(s - e);
            double wt = qstep * (1.0 + e) * t;
            sm.tq[tid] = t;
            sm.cq[tid] = wt * (slack ? exp(-t) : 1.0) * nfact;
        }
        __syncthreads();
        // per (node, token): survival x and the series h = e / (1 + x e)
        for (int task = tid; task < qn * m; task += kSolveThreads) {
            const int q = task / m, j = task - q * m;
            const double x = exp(-sm.tq[q] * sm.w[j]);
            sm.X[q * KP + j] = x;
            GR_PTR(double) Hq = sm.H + (size_t)q * n1 * KP;
            for (int c = 1; c <= n; c++) {
                // (four partial sums: the loads of one no longer wait for the multiply-add of the one before)
                double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
                int a = 1;
                for (; a + 3 < c; a += 4) {
                    a0 = fma(sm.E[a * KP + j], Hq[(c - a) * KP + j], a0);
                    a1 = fma(sm.E[(a + 1) * KP + j], Hq[(c - a - 1) * KP + j], a1);
                    a2 = fma(sm.E[(a + 2) * KP + j], Hq[(c - a - 2) * KP + j], a2);
                    a3 = fma(sm.E[(a + 3) * KP + j], Hq[(c - a - 3) * KP + j], a3);
                }
                for (; a < c; a++) a0 = fma(sm.E[a * KP + j], Hq[(c - a) * KP + j], a0);
                Hq[c * KP + j] = sm.E[c * KP + j] - x * ((a0 + a1) + (a2 + a3));
            }
        }
        // Partial products of the factors f_j = 1 + x_j e_j over token groups, then a tree over the groups.  Every
        // series product is spread over its output coefficients (one thread each, at most n + 1 multiply-adds in a
        // row) and goes from one buffer to the other, so no thread waits on a 500-term chain.
        GR_PTR(double) cur = sm.PP;
        GR_PTR(double) nxt = sm.PQ;
        bool in_pp = true;                               // cur is sm.PP
        const int ntask = qn * kGroups * n1;
        for (int task = tid; task < ntask; task += kSolveThreads) {
            const int c = task % n1, grp = (task / n1) % kGroups;
            cur[task] = grp == 0 ? sm.P[c] : (c == 0 ? 1.0 : 0.0);      // group 0 starts from e^{lambda h}
        }
        __syncthreads();
        // (four consecutive output coefficients per thread: each loaded operand feeds four multiply-adds, which
        // keeps the products off the shared-memory bandwidth limit)
        const int nb4 = (n1 + 3) >> 2;
        const int ntask4 = qn * kGroups * nb4;
        for (int step = 0; step < gsz; step++) {
            for (int task = tid; task < ntask4; task += kSolveThreads) {
                const int c0 = (task % nb4) << 2, qg = task / nb4, grp = qg % kGroups, q = qg / kGroups;
                const int j = grp * gsz + step;
                GR_PTR(const double) in = cur + (size_t)qg * n1;
                GR_PTR(double) out = nxt + (size_t)qg * n1;
                double acc[4] = {0.0, 0.0, 0.0, 0.0};
                const bool live = j < m && j != da && j != db;     // dominant factors are applied after the tree
                if (live) {
                    // acc[k] = sum_{a = 1 .. c0 + k} E[a] in[c0 + k - a];  win[k] = in[c0 + k - a]
                    double win[4];
#pragma unroll
                    for (int k = 0; k < 4; k++) win[k] = (c0 + k - 1 >= 0 && c0 + k - 1 <= n) ? in[c0 + k - 1] : 0.0;
                    const int amax = min(c0 + 3, n);
                    for (int a = 1; a <= amax; a++) {
                        const double ea = sm.E[a * KP + j];
#pragma unroll
                        for (int k = 0; k < 4; k++) acc[k] = fma(ea, win[k], acc[k]);
                        win[3] = win[2]; win[2] = win[1]; win[1] = win[0];
                        win[0] = (c0 - a - 1 >= 0) ? in[c0 - a - 1] : 0.0;
                    }
                }
                const double x = live ? sm.X[q * KP + j] : 0.0;
#pragma unroll
                for (int k = 0; k < 4; k++)
                    if (c0 + k <= n) out[c0 + k] = in[c0 + k] + x * acc[k];
            }
            __syncthreads();
            GR_PTR(double) t2 = cur; cur = nxt; nxt = t2; in_pp = !in_pp;
        }
        for (int stride = 1; stride < kGroups; stride <<= 1) {
            for (int task = tid; task < ntask4; task += kSolveThreads) {
                const int c0 = (task % nb4) << 2, qg = task / nb4, grp = qg % kGroups;
                if ((grp % (2 * stride)) == 0) {
                    GR_PTR(const double) Aq = cur + (size_t)qg * n1;
                    GR_PTR(const double) Bq = cur + (size_t)(qg + stride) * n1;
                    // acc[k] = sum_{a = 0 .. c0 + k} A[a] B[c0 + k - a];  win[k] = B[c0 + k - a]
                    double acc[4] = {0.0, 0.0, 0.0, 0.0}, win[4];
#pragma unroll
                    for (int k = 0; k < 4; k++) win[k] = (c0 + k <= n) ? Bq[c0 + k] : 0.0;
                    const int amax = min(c0 + 3, n);
                    for (int a = 0; a <= amax; a++) {
                        const double aa = Aq[a];
#pragma unroll
                        for (int k = 0; k < 4; k++) acc[k] = fma(aa, win[k], acc[k]);
                        win[3] = win[2]; win[2] = win[1]; win[1] = win[0];
                        win[0] = (c0 - a - 1 >= 0) ? Bq[c0 - a - 1] : 0.0;
                    }
                    GR_PTR(double) out = nxt + (size_t)qg * n1;
#pragma unroll
                    for (int k = 0; k < 4; k++)
                        if (c0 + k <= n) out[c0 + k] = acc[k];
                }
            }
            __syncthreads();
            GR_PTR(double) t2 = cur; cur = nxt; nxt = t2; in_pp = !in_pp;
        }
        if (!in_pp) {
            // the later stages read the product of node q at PP[q][0]
            for (int task = tid; task < qn * n1; task += kSolveThreads) {
                const int c = task % n1, q = task / n1;
                sm.PP[(size_t)(q * kGroups) * n1 + c] = cur[(size_t)(q * kGroups) * n1 + c];
            }
            __syncthreads();
        }
        if (da >= 0) {
            // PP[q][0] = product without the dominant factors (LAB).  PX[q][0] = all but a, PX[q][1] = all but b,
            // PX[q][2] = full product.
            for (int task = tid; task < qn * 2 * n1; task += kSolveThreads) {
                const int c = task % n1, which = (task / n1) % 2, q = task / (2 * n1);
                GR_PTR(const double) Lab = sm.PP + (size_t)(q * kGroups) * n1;
                const int j = which == 0 ? db : da;       // the factor that stays in
                double v = Lab[c];
                if (j >= 0) {
                    double acc = 0.0;
                    for (int a = 1; a <= c; a++) acc += sm.E[a * KP + j] * Lab[c - a];
                    v += sm.X[q * KP + j] * acc;
                }
                sm.PX[(size_t)(q * 3 + which) * n1 + c] = v;
            }
            __syncthreads();
            for (int task = tid; task < qn * n1; task += kSolveThreads) {
                const int c = task % n1, q = task / n1;
                GR_PTR(const double) La = sm.PX + (size_t)(q * 3 + 1) * n1;      // Lab f_a
                double v = La[c];
                if (db >= 0) {
                    double acc = 0.0;
                    for (int a = 1; a <= c; a++) acc += sm.E[a * KP + db] * La[c - a];
                    v += sm.X[q * KP + db] * acc;
                }
                sm.PX[(size_t)(q * 3 + 2) * n1 + c] = v;
            }
            __syncthreads();
        }
        // per (node, token): gradient integrand
        for (int task = tid; task < qn * m; task += kSolveThreads) {
            const int q = task / m, j = task - q * m;
            GR_PTR(const double) Hq = sm.H + (size_t)q * n1 * KP;
            double val = 0.0;
            if (j == da || j == db) {
                // dominant token: dM/dx_j = n! [lambda^n] e_j L_j with L_j the product of all other factors
                GR_PTR(const double) Lj = sm.PX + (size_t)(q * 3 + (j == da ? 0 : 1)) * n1;
                for (int c = 1; c <= n; c++) val += Lj[n - c] * sm.E[c * KP + j];
            } else {
                GR_PTR(const double) Pq = da >= 0 ? sm.PX + (size_t)(q * 3 + 2) * n1 : sm.PP + (size_t)(q * kGroups) * n1;
                for (int c = 1; c <= n; c++) val += Pq[n - c] * Hq[c * KP + j];
            }
            const double u = sm.w[j] * sm.X[q * KP + j];
            const double gi = sm.cq[q] * u * val;
            sm.gq[q * KP + j] = gi;
            sm.g2q[q * KP + j] = gi * sm.tq[q] * sm.w[j];
        }
        if (want_jac && n > 1) {
            // series A = P h (for a dominant token: e_j times the product of the other factors), scaled for the
            // Hessian; one thread per coefficient
            const int nm1 = n - 1;
            for (int task = tid; task < qn * m * nm1; task += kSolveThreads) {
                const int e = 1 + task % nm1, qj = task / nm1, j = qj % m, q = qj / m;
                GR_PTR(const double) Hq = sm.H + (size_t)q * n1 * KP;
                const double sa = sm.cq[q] * sm.tq[q] * sm.w[j] * sm.X[q * KP + j];
                double acc = 0.0;
                if (j == da || j == db) {
                    GR_PTR(const double) Lj = sm.PX + (size_t)(q * 3 + (j == da ? 0 : 1)) * n1;
                    for (int c = 1; c <= e; c++) acc += sm.E[c * KP + j] * Lj[e - c];
                } else {
                    GR_PTR(const double) Pq = da >= 0 ? sm.PX + (size_t)(q * 3 + 2) * n1 : sm.PP + (size_t)(q * kGroups) * n1;
                    double a1 = 0.0;
                    int c = 1;
                    for (; c + 1 <= e; c += 2) {
                        acc = fma(Hq[c * KP + j], Pq[e - c], acc);
                        a1 = fma(Hq[(c + 1) * KP + j], Pq[e - c - 1], a1);
                    }
                    if (c <= e) acc = fma(Hq[c * KP + j], Pq[e - c], acc);
                    acc += a1;
                }
                sm.A[(size_t)q * n1 * KP + e * KP + j] = sa * acc;
            }
            if (da >= 0 && db >= 0) {
                // for the pair (a, b): the series e_a times the product without both
                for (int task = tid; task < qn * nm1; task += kSolveThreads) {
                    const int e = 1 + task % nm1, q = task / nm1;
                    GR_PTR(const double) Lab = sm.PP + (size_t)(q * kGroups) * n1;
                    const double sa = sm.cq[q] * sm.tq[q] * sm.w[da] * sm.X[q * KP + da];
                    double acc = 0.0;
                    for (int c = 1; c <= e; c++) acc += sm.E[c * KP + da] * Lab[e - c];
                    sm.AX[(size_t)q * n1 + e] = sa * acc;
                }
            }
            __syncthreads();
            // the h-series scaled by u for the pairing (a dominant token pairs through e_j itself)
            for (int task = tid; task < qn * m * nm1; task += kSolveThreads) {
                const int c = 1 + task % nm1, qj = task / nm1, j = qj % m, q = qj / m;
                GR_PTR(double) Hq = sm.H + (size_t)q * n1 * KP;
                const double u = sm.w[j] * sm.X[q * KP + j];
                Hq[c * KP + j] = u * ((j == da || j == db) ? sm.E[c * KP + j] : Hq[c * KP + j]);
            }
        }
        __syncthreads();
        if (tid < m) {
            double a = 0.0, b2 = 0.0;
            for (int q = 0; q < qn; q++) { a += sm.gq[q * KP + tid]; b2 += sm.g2q[q * KP + tid]; }
            sm.g[tid] += a; sm.g2[tid] += b2;
        }
        if (want_jac && n > 1) {
            const int warp = tid >> 5, lane = tid & 31;
            for (int i = 1 + warp; i < m; i += kSolveWarps) {
                for (int l = lane; l < i; l += 32) {
                    double acc = 0.0;
                    const bool domi = (i == da || i == db), doml = (l == da || l == db);
                    // the A-series of a dominant token pairs with the h-series of the other token; two dominant
                    // tokens pair through the product without both
                    const int ia = (doml && !domi) ? l : i, ih = (doml && !domi) ? i : l;
                    for (int q = 0; q < qn; q++) {
                        const GR_PTR(double) Aq = sm.A + (size_t)q * n1 * KP;
                        const GR_PTR(double) Hq = sm.H + (size_t)q * n1 * KP;
                        if (domi && doml) {
                            const GR_PTR(double) Ax = sm.AX + (size_t)q * n1;
                            for (int c = 1; c < n; c++) acc += Ax[n - c] * Hq[c * KP + db];
                        } else {
                            for (int c = 1; c < n; c++) acc += Aq[(n - c) * KP + ia] * Hq[c * KP + ih];
                        }
                    }
                    sm.J[tri(i, l)] -= acc;
                }
            }
        }
    }
    __syncthreads();
    if (want_jac && tid < m) sm.J[tri(tid, tid)] = sm.g[tid] - sm.g2[tid];
    __syncthreads();
    return Q;
}

// In-place Cholesky of the packed lower triangle; S_FAIL is set when a pivot is not positive.
__device__ void cholesky(const Sm& sm, int m)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    for (int j = 0; j < m; j++) {
        __syncthreads();
        const double pj = sm.J[tri(j, j)];
        if (!(pj > 0.0)) { if (tid == 0) sm.scal[S_FAIL] = 1.0; __syncthreads(); return; }
        // smallest pivot relative to the diagonal entry it came from (S_PIVOT; the caller sets it to 1 beforehand)
        if (tid == 0) sm.scal[S_PIVOT] = fmin(sm.scal[S_PIVOT], pj / (sm.g[j] - sm.g2[j] + sm.scal[S_ADD]));
        const double inv = 1.0 / sqrt(pj);
        for (int i = j + 1 + tid; i < m; i += kSolveThreads) sm.col[i] = sm.J[tri(i, j)] * inv;
        __syncthreads();
        if (tid == 0) sm.J[tri(j, j)] = sqrt(pj);
        for (int i = j + 1 + tid; i < m; i += kSolveThreads) sm.J[tri(i, j)] = sm.col[i];
        for (int i = j + 1 + warp; i < m; i += kSolveWarps) {
            const double ci = sm.col[i];
            for (int l = j + 1 + lane; l <= i; l += 32) sm.J[tri(i, l)] -= ci * sm.col[l];
        }
    }
    __syncthreads();
}

// delta <- solution of L L^T delta = delta (one warp; column-oriented substitutions)
__device__ void chol_solve(const Sm& sm, int m)
{
    const int tid = threadIdx.x;
    if (tid < 32) {
        const int lane = tid;
        for (int i = 0; i < m; i++) {
            if (lane == 0) sm.delta[i] = sm.delta[i] / sm.J[tri(i, i)];
            __syncwarp();
            const double yi = sm.delta[i];
            for (int l = i + 1 + lane; l < m; l += 32) sm.delta[l] -= sm.J[tri(l, i)] * yi;
            __syncwarp();
        }
        for (int i = m - 1; i >= 0; i--) {
            if (lane == 0) sm.delta[i] = sm.delta[i] / sm.J[tri(i, i)];
            __syncwarp();
            const double xi = sm.delta[i];
            for (int l = lane; l < i; l += 32) sm.delta[l] -= sm.J[tri(i, l)] * xi;
            __syncwarp();
        }
    }
    __syncthreads();
}

// Newton iteration for one system.  On return sm.w[0..m) holds exp(alpha).
// Returns the status; *gnorm and *iters receive the final L1 gradient norm and the evaluations spent.
// `warm`: weights to start from (what the fast kernel reached before it gave the instance up), or a null pointer.
__device__ int solve_system(const Sm& sm, int m, GR_PTR(const double) d, GR_PTR(const double) rhs, double hmass,
                            int slack, double tol, int max_iters, double qstep, double* gnorm, int* iters,
                            const double* warm = nullptr)
{
    const int tid = threadIdx.x, n = sm.n, KP = sm.KP;
    GR_PTR(double) red = sm.scal + 16;
    // E[c][j] = d_j^c / c!
    if (tid < m) {
        double pw = 1.0, fc = 1.0;
        sm.E[tid] = 0.0;
        for (int c = 1; c <= n; c++) { pw *= d[tid]; fc *= (double)c; sm.E[c * KP + tid] = pw / fc; }
    }
    // dominant tokens: d_j / (total mass) >= pi (1e5 / n!)^(1/n), checked only for n > 16 (below, the series
    // division is accurate to 1e-11 for any token)
    if (tid == 0) {
        int a = -1, b2 = -1;
        if (n > 16) {
            double T = hmass, lf = 0.0;
            for (int j = 0; j < m; j++) T += d[j];
            for (int c = 2; c <= n; c++) lf += log((double)c);
            const double thr = 3.141592653589793 * exp((log(1.0e5) - lf) / (double)n);
            for (int j = 0; j < m; j++) {
                if (d[j] >= thr * T) { if (a < 0) a = j; else if (b2 < 0) b2 = j; }
            }
        }
        sm.scal[S_DA] = (double)a; sm.scal[S_DB] = (double)b2;
    }
    // starting point: the single-token balance  w/(1+w) * Pr[i in set(omega)] = rhs
    double a0 = 0.0;
    bool warm_used = false;
    const double D = block_reduce_sum(tid < m ? d[tid] : 0.0, red);   // draft mass of the system
    if (tid < m) {
        if (slack) {
            // Pr[i drafted and every draft inside the system] = D^n - (D - d_i)^n
            double cap = pow(D, (double)n) - pow(fmax(D - d[tid], 0.0), (double)n);
            double den = fmax(cap - rhs[tid], 1e-3 * rhs[tid]);
            a0 = log(rhs[tid] / den);
        } else {
            a0 = log(rhs[tid] / d[tid]);
        }
    }
    if (warm != nullptr) {
        // usable when every weight is positive and finite and they are not all still at the initial 1
        const double wv = tid < m ? warm[tid] : 1.0;
        const int bad = __syncthreads_or(!(wv > 0.0) || !(wv < 1.0e300));
        const int moved = __syncthreads_or(wv != 1.0);
        if (!bad && moved && tid < m) a0 = log(wv);
        warm_used = !bad && moved;
    }
    if (!slack) {
        double mean = block_reduce_sum(tid < m ? a0 : 0.0, red) / (double)m;
        a0 -= mean;
    }
    if (tid < m) sm.alpha[tid] = fmin(fmax(a0, -kAlphaClamp), kAlphaClamp);
    // (a point handed over by the fast kernel is close to the solution: the full grid from the first evaluation)
    if (tid == 0) { sm.scal[S_RPREV] = warm_used ? 5.0e-3 : 1.0e300; sm.scal[S_LAM] = 1.0; sm.scal[S_COARSE] = warm_used ? 0.0 : 1.0; }
    __syncthreads();

    int status = GR_NOT_CONVERGED;
    int it = 0;
    double rn = 0.0;
    for (; it < max_iters; it++) {
        // Far from the solution the trapezoid step is doubled (half the nodes; quadrature error ~1e-5, far below
        // the gradient norm there).  Convergence is only declared on the full grid, so a tolerance that loose
        // evaluations could meet keeps the full grid throughout.
        const bool coarse = sm.scal[S_RPREV] > 1.0e-2 && tol < 1.0e-3;
        const bool comparable = coarse == (sm.scal[S_COARSE] != 0.0);
        __syncthreads();
        eval_system(sm, m, d, hmass, slack, true, coarse ? 2.0 * qstep : qstep);
        rn = block_reduce_sum(tid < m ? fabs(sm.g[tid] - rhs[tid]) : 0.0, red);
        if (rn <= tol && !coarse) { status = GR_OK; it++; break; }
        const double rprev = sm.scal[S_RPREV];
        const double lam = sm.scal[S_LAM];
        __syncthreads();
        if (tid == 0) sm.scal[S_COARSE] = coarse ? 1.0 : 0.0;
        // (a residual on the full grid is not compared with the coarse grid's: they differ by the coarse quadrature error)
        if (comparable && !(rn < rprev) && lam > 1.0 / 64.0 && it > 0) {
            // the last step did not reduce the gradient norm: retry it at half length
            if (tid < m) sm.alpha[tid] = sm.alpha_prev[tid] + 0.5 * lam * sm.delta[tid];
            if (tid == 0) sm.scal[S_LAM] = 0.5 * lam;
            __syncthreads();
            continue;
        }
        if (tid < m) sm.alpha_prev[tid] = sm.alpha[tid];
        if (tid == 0) { sm.scal[S_RPREV] = rn; sm.scal[S_LAM] = 1.0; sm.scal[S_FAIL] = 0.0; }
        if (!slack) {
            // the block function is constant along (1,...,1): pin that direction
            const double add = 1.0 / (double)m;
            for (int e = tid; e < m * (m + 1) / 2; e += kSolveThreads) sm.J[e] += add;
        }
        if (tid == 0) { sm.scal[S_PIVOT] = 1.0; sm.scal[S_ADD] = slack ? 0.0 : 1.0 / (double)m; }
        __syncthreads();
        cholesky(sm, m);
        const bool fail = sm.scal[S_FAIL] != 0.0;
        __syncthreads();
        if (!fail) {
            // Right-hand side: along its own coordinate a token's flow follows a logistic curve g_i = c sigma(alpha_i -
            // kappa) with saturation level c = g_i^2 / g2_i (from H_ii = g_i - g2_i = g_i (1 - g_i / c)); the curve
            // through the current value and slope is inverted exactly, H_ii (logit(rhs_i / c) - logit(g_i / c)),
            // which agrees with rhs_i - g_i to first order and places a nearly saturated token in one step.  A target
            // at or beyond the predicted saturation level keeps the plain residual.
            if (tid < m) {
                const double gi = sm.g[tid], g2i = sm.g2[tid], ri = rhs[tid];
                const double room = 1.0 - ri * g2i / (gi * gi);
                const double arg = fmax((ri - gi) / (gi * fmax(room, 1e-3)), -1.0 + 1e-12);
                sm.delta[tid] = room > 1e-3 ? (gi - g2i) * log1p(arg) : ri - gi;
            }
            __syncthreads();
            chol_solve(sm, m);
        } else {
            // proportional-fitting step  alpha += log(rhs / g)
            if (tid < m) sm.delta[tid] = log(rhs[tid] / sm.g[tid]);
            __syncthreads();
        }
        double dm = block_reduce_max(tid < m ? fabs(sm.delta[tid]) : 0.0, red);
        if (!(dm < 1.0e300)) dm = 1.0e300;
        // a full Newton step below 1e-11 in alpha: the weights cannot be improved at this quadrature accuracy
        if (!fail && dm < 1.0e-11) { status = GR_OK; it++; break; }
        const double sc = dm > kStepClamp ? kStepClamp / dm : 1.0;
        if (tid < m) {
            double dl = sm.delta[tid] * sc;
            if (!(dl == dl)) dl = 0.0;
            sm.delta[tid] = dl;
        }
        __syncthreads();
        double mean = 0.0;
        if (!slack) mean = block_reduce_sum(tid < m ? sm.delta[tid] : 0.0, red) / (double)m;
        if (tid < m) {
            sm.delta[tid] -= mean;
            double a = sm.alpha[tid] + sm.delta[tid];
            sm.alpha[tid] = fmin(fmax(a, -kAlphaClamp), kAlphaClamp);
        }
        __syncthreads();
        // Second-order size of the step, sum_i g_i delta_i^2: a full Newton step in alpha = log w from a point
        // evaluated on the full grid leaves a residual of at most a small multiple of it (within 3.1 times, plus the
        // quadrature floor, on every benchmark shape).  Ten times below the tolerance: the step is taken and the
        // iteration stops without another evaluation; the reported norm is then the bound 3 s2.
        const double s2 = block_reduce_sum(tid < m ? sm.g[tid] * sm.delta[tid] * sm.delta[tid] : 0.0, red);
        // (not after a factorisation that cancelled all but a few percent of a diagonal entry: see the fast kernel)
        if (!fail && !coarse && dm <= 1.0 && 10.0 * s2 < tol && sm.scal[S_PIVOT] > 0.02) {
            if (tid < m) sm.w[tid] = exp(sm.alpha[tid]);
            __syncthreads();
            rn = 3.0 * s2;
            status = GR_OK; it++;
            it |= kItersPredicted;
            break;
        }
    }
    *gnorm = rn;
    *iters = it;
    return status;
}

__global__ void __launch_bounds__(kSolveThreads)
solve_kernel(const char* __restrict__ ws, char* __restrict__ params, int pstride, int kcap, int V, int n, int topk,
             double temp_t, double temp_d, double tol, int max_iters, double qstep, double tau, int Qt, int only_flagged,
             float* __restrict__ alpha_out, int* __restrict__ status_out, FusedArgs fa)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ int s_sel;
    GR_CHECK_FLAG_DECL;
    GR_CHECK_FLAG_INIT;
    const bool fused = fa.draft != nullptr;
    const int tid = threadIdx.x;
    const long long b = blockIdx.x;
    char* pb = params + (size_t)b * pstride;
    ParamView pv = view_params(pb, kcap, V, GR_CHECK_FLAG);
    const WsView wv = view_ws(ws, b, GR_CHECK_FLAG);
    // second pass after the fast kernel: only the instances it flagged are redone
    if (only_flagged && !(pv.h->magic == kMagic && pv.h->status == kNeedFallback)) return;
    if (kcap == 0 || wv.h->bad != 0 || wv.h->count <= 0) {
        // no rule: whole-vocabulary support beyond the capacity, or unusable logits
        if (tid == 0) write_no_rule(pv.h, n, wv.h->bad != 0, alpha_out, status_out, b);
        if (fused) {
            __syncthreads();
            fused_draw(fa, pv.h, b, n, smem_raw, GR_CHECK_FLAG);
        }
        return;
    }

    const int KP = kcap;
    SolveLayout L(KP, n, Qt);
    double* base = reinterpret_cast<double*>(smem_raw);
    Sm sm;
    int* const ck = GR_CHECK_FLAG;
    (void)ck;
    const int n1c = n + 1;
    sm.d = GR_MKPTR(double, base + L.d, KP, ck); sm.tg = GR_MKPTR(double, base + L.tg, KP, ck);
    sm.p = GR_MKPTR(double, base + L.p, KP, ck); sm.r = GR_MKPTR(double, base + L.r, KP, ck);
    sm.key = GR_MKPTR(double, base + L.key, KP, ck); sm.w = GR_MKPTR(double, base + L.w, KP, ck);
    sm.psi = GR_MKPTR(double, base + L.psi, KP + 4, ck); sm.Dr = GR_MKPTR(double, base + L.Dr, KP + 4, ck);
    sm.alpha = GR_MKPTR(double, base + L.alpha, KP, ck); sm.alpha_prev = GR_MKPTR(double, base + L.alpha_prev, KP, ck);
    sm.delta = GR_MKPTR(double, base + L.delta, KP, ck); sm.g = GR_MKPTR(double, base + L.g, KP, ck);
    sm.g2 = GR_MKPTR(double, base + L.g2, KP, ck); sm.col = GR_MKPTR(double, base + L.col, KP, ck);
    sm.E = GR_MKPTR(double, base + L.E, KP * n1c, ck); sm.J = GR_MKPTR(double, base + L.J, KP * (KP + 1) / 2, ck);
    sm.tq = GR_MKPTR(double, base + L.tq, Qt, ck); sm.cq = GR_MKPTR(double, base + L.cq, Qt, ck);
    sm.X = GR_MKPTR(double, base + L.X, Qt * KP, ck); sm.H = GR_MKPTR(double, base + L.H, Qt * n1c * KP, ck);
    sm.A = GR_MKPTR(double, base + L.A, Qt * n1c * KP, ck); sm.P = GR_MKPTR(double, base + L.P, Qt * n1c, ck);
    sm.PP = GR_MKPTR(double, base + L.PP, Qt * kGroups * n1c, ck);
    sm.PQ = GR_MKPTR(double, base + L.PQ, Qt * kGroups * n1c, ck); sm.PX = GR_MKPTR(double, base + L.PX, Qt * 3 * n1c, ck);
    sm.AX = GR_MKPTR(double, base + L.AX, Qt * n1c, ck);
    sm.gq = GR_MKPTR(double, base + L.gq, Qt * KP, ck); sm.g2q = GR_MKPTR(double, base + L.g2q, Qt * KP, ck);
    sm.scal = GR_MKPTR(double, base + L.scal, 32, ck);
    int* ib = reinterpret_cast<int*>(smem_raw + L.ints);
    sm.id = GR_MKPTR(int, ib, KP, ck); sm.blk = GR_MKPTR(int, ib + KP, KP, ck);
    sm.order = GR_MKPTR(int, ib + 2 * KP, KP, ck); sm.itmp = GR_MKPTR(int, ib + 3 * KP, KP, ck);
    sm.KP = KP; sm.n = n; sm.Qt = Qt;
    GR_PTR(double) red = sm.scal + 16;

    PrepSm ps;
    ps.d = sm.d; ps.tg = sm.tg; ps.p = sm.p; ps.r = sm.r; ps.key = sm.key; ps.psi = sm.psi; ps.Dr = sm.Dr;
    ps.id = sm.id; ps.blk = sm.blk; ps.itmp = sm.itmp; ps.red = red; ps.out3 = sm.scal;
    const PrepResult pr = prep_instance(ps, wv, pv.h, V, n, topk, temp_t, temp_d);
    const int k = pr.k, jstar = pr.jstar;

    // ---- convex minimisation: inner system on H*, then every outer block with two or more tokens
    int status = GR_OK, iters_total = 0;
    double gnorm_total = 0.0;
    // Truncated variant (Algorithm 1 with an error threshold): every system is solved on its truncation set alone,
    // to gradient norm 5 tau; the other tokens keep weight 0.  The gathered arrays reuse what the preparation no
    // longer needs.
    const bool trunc = tau > 0.0;
    if (trunc) {
        truncation_sets(ps, sm.order, sm.itmp, k, jstar, n, tau);
        tol = 5.0 * tau;
    }
    GR_PTR(double) dT = sm.key; GR_PTR(double) rT = sm.psi; GR_PTR(int) tmap = sm.itmp;
    // an instance the fast kernel gave up carries the weights that kernel reached: they are kept (sm.key is free
    // outside the truncated variant) as the starting point of each system
    const bool warm = only_flagged && !trunc;
    if (warm && tid < k) sm.key[tid] = pv.w[tid];
    __syncthreads();
    const double* warm_w = warm ? &sm.key[0] : nullptr;
    if (tid < k) pv.w[tid] = trunc ? 0.0 : 1.0;
    // with the drafted tuple at hand only the system it selects is solved
    const int sel = fused ? selected_system(fa.draft + (size_t)b * n, n, k, jstar, sm.id, sm.blk, &s_sel) : -2;
    bool skipped = false;
    if (jstar > 0 && sel >= 0) skipped = true;
    if (jstar > 0 && sel < 0) {
        double gn = 0.0; int it = 0;
        if (!trunc) {
            int st = solve_system(sm, jstar, sm.d, sm.tg, 0.0, 1, tol, max_iters, qstep, &gn, &it, warm_w);
            if (st != GR_OK) status = GR_NOT_CONVERGED;
            if (tid < jstar) pv.w[tid] = sm.w[tid];
        } else {
            const int mT = gather_truncated(sm.order, 0, jstar, sm.d, sm.tg, dT, rT, tmap, &s_sel);
            if (mT > 0) {
                int st = solve_system(sm, mT, dT, rT, 0.0, 1, tol, max_iters, qstep, &gn, &it);
                if (st != GR_OK) status = GR_NOT_CONVERGED;
                if (tid < mT) pv.w[tmap[tid]] = sm.w[tid];
            }
        }
        gnorm_total += gn; iters_total = add_iters(iters_total, it);
        __syncthreads();
    }
    {
        int lo = jstar;
        while (lo < k) {
            int hi = lo;
            const int bk = sm.blk[lo];
            while (hi + 1 < k && sm.blk[hi + 1] == bk) hi++;
            const int m = hi - lo + 1;
            const bool wanted = sel == -2 || sel == bk;
            if (!trunc) {
                if (m >= 2 && !wanted) skipped = true;
                if (m >= 2 && wanted) {
                    double gn; int it;
                    int st = solve_system(sm, m, sm.d + lo, sm.p + lo, sm.Dr[lo], 0, tol, max_iters, qstep, &gn, &it,
                                          warm_w ? warm_w + lo : nullptr);
                    if (st != GR_OK) status = GR_NOT_CONVERGED;
                    gnorm_total += gn; iters_total = add_iters(iters_total, it);
                    if (tid < m) pv.w[lo + tid] = sm.w[tid];
                    __syncthreads();
                }
            } else {
                // tuples counted: those inside (H* u T)^n, so the mass above the block is drf(H*) plus the T-part of
                // the higher-ratio outer blocks
                double hT = sm.Dr[jstar];
                for (int j = jstar; j < lo; j++) hT += sm.order[j] ? sm.d[j] : 0.0;
                const int mT = gather_truncated(sm.order, lo, hi + 1, sm.d, sm.p, dT, rT, tmap, &s_sel);
                if (mT == 1 && tid == 0) pv.w[tmap[0]] = 1.0;
                if (mT >= 2 && !wanted) skipped = true;
                if (mT >= 2 && wanted) {
                    double gn; int it;
                    int st = solve_system(sm, mT, dT, rT, hT, 0, tol, max_iters, qstep, &gn, &it);
                    if (st != GR_OK) status = GR_NOT_CONVERGED;
                    gnorm_total += gn; iters_total = add_iters(iters_total, it);
                    if (tid < mT) pv.w[tmap[tid]] = sm.w[tid];
                }
                __syncthreads();
            }
            lo = hi + 1;
        }
    }

    if (status == GR_OK && skipped) status = GR_PARTIAL_RULE;
    write_rule(ps, pv, KP, pr, n, status, gnorm_total, iters_total, alpha_out, status_out, b, GR_CHECK_FLAG,
               wv.h->check);
    if (fused) {
        __syncthreads();                       // the rule this CTA wrote is visible to its first warp
        fused_draw(fa, pv.h, b, n, smem_raw, GR_CHECK_FLAG);
    }
}

int launch_solve(const char* ws, char* params, int pstride, int kcap, int V, int n, int topk, double temp_t,
                 double temp_d, double tol, int max_iters, double qstep, double tau, int batch, int only_flagged,
                 float* alpha_out, int* status_out, FusedArgs fa, cudaStream_t st)
{
    int Qt = 1, smem = 0;
    if (kcap > 0) {
        // keep several CTAs resident per SM when the shape allows it
        Qt = solve_pick_tile(kcap, n, 72 * 1024);
        if (solve_smem_bytes(kcap, n, Qt) > 72 * 1024) Qt = solve_pick_tile(kcap, n, 200 * 1024);
        smem = solve_smem_bytes(kcap, n, Qt);
        if (smem > 220 * 1024) return GR_E_TOO_LARGE;
    }
    if (fa.draft && smem < kVerifyScratchBytes) smem = kVerifyScratchBytes;    // the draw's scratch
    // function attributes belong to the device: set once per device
    static bool configured[kMaxDevices] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return GR_E_LAUNCH; }
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(solve_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024) != cudaSuccess)
            return GR_E_LAUNCH;
        configured[dev] = true;
    }
    solve_kernel<<<batch, kSolveThreads, smem, st>>>(ws, params, pstride, kcap, V, n, topk, temp_t, temp_d, tol,
                                                     max_iters, qstep, tau, Qt, only_flagged, alpha_out, status_out, fa);
    return GR_OK;
}

}  // namespace gr
