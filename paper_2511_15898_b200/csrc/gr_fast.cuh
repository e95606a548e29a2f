// Fast per-instance solve for supports up to 128 tokens and n <= 16: one CTA per instance, 96 threads and four
// CTAs per SM for supports up to 64, 128 threads and one CTA per SM above.
//
// Same mathematics as the robust kernel (gr_solve.cu): the gradient of the convex functions
// of the inner system / of an outer block (Thm "Inner Convex Solver", Thm "Outer Convex Solver")
// is the one-dimensional integral
//   g_i = w_i int e^{-t slack} x_i(t) n! [lambda^n] P(lambda; t) h_i(lambda; t) dt,
// and Newton's method on alpha = log w uses its exact Hessian.  Organised for throughput:
//   - one warp per quadrature node, one lane per token (up to four tokens per lane on the larger supports):
//     every power series lives in registers;
//   - the product P = e^{lambda h} prod_j f_j over the tokens is not multiplied out:
//     d/dlambda log f_j = x_j d_j (1 + (1 - x_j) h_j), so the log-derivative S of P is a SUM over
//     tokens (a warp reduction) and P follows from P' = S P.  In fp64 this is accurate to
//     ~1e-12 for n <= 16 and degrades beyond (larger n takes the robust kernel);
//   - h_j(lambda) = H(d_j lambda; x_j) with H(mu; x) = (e^mu - 1) / (1 + x (e^mu - 1)), whose
//     coefficients obey a recurrence with compile-time constants 1/c!;
//   - the Hessian's off-diagonal part  - sum_q c_q t_q (w x)_i (w x)_l n! [lambda^n] P h_i h_l  is a
//     dense contraction over (node, series index); it only steers the iteration, so it is
//     taken on every second node (trapezoid step doubled) and accumulated in fp32 from operands
//     staged in shared memory; the gradient itself stays fp64 on every node;
//   - the iteration starts from a mean-field point (each token against the expected weight
//     of the other drafted tokens, with a bound on what a single huge competitor can add).
#pragma once
#include "gr_prep.cuh"
#include "gr_verify.cuh"

// The translation unit that includes this file chooses the padded support size: 64 (96-thread CTAs, four per
// SM) or 128 (256-thread CTAs, one per SM: its shared memory admits no second CTA, so the one CTA brings two warps
// per scheduler itself), and a namespace of its own for the instantiation.
#ifndef GR_FAST_MP
#define GR_FAST_MP 64
#define GR_FAST_NS fast64
#endif

namespace gr {
namespace GR_FAST_NS {

constexpr int kMP = GR_FAST_MP;       // padded support size of these kernels
constexpr int kRL = kMP / 32;         // rows (or tokens) per lane when a warp covers the whole support
constexpr int kFT = kMP == 64 ? 96 : 256;   // threads per CTA (at least kMP - 8: one thread per panel row)
constexpr int kFCtas = kMP == 64 ? 4 : 1;   // CTAs per SM the kernels are compiled for
constexpr int kFW = kFT / 32;         // warps per CTA
constexpr int kJC = kMP == 64 ? 6 : 4;      // Hessian nodes staged per chunk
constexpr double kFTEnd = 25.0;       // quadrature range constants, identical to the robust kernel's
constexpr double kFDrop = 1.0;
constexpr double kFTail = 3.0;
constexpr int kFMaxNodes = 128;
constexpr int kMS = kMP + 8;          // row stride of the staged operands (floats): conflict-free MMA fragment loads
constexpr int kJS = kMP + 1;          // row stride of the contraction accumulator / Hessian (floats)
constexpr double kFAlphaClamp = 80.0;
constexpr double kFStepClamp = 3.0;
constexpr double kFPredictStep = 1.0;      // largest |delta alpha| after which the stop on a predicted residual is allowed
constexpr double kFPredictSafety = 10.0;   // the prediction s2 must be this many times below the tolerance
constexpr double kFRatioSafety = 3.0;      // the predicted residual rho * r must be this many times below the tolerance
constexpr double kFTrustPivot = 0.02;       // smallest relative pivot at which a predicted stop is allowed
constexpr double kFPredictBound = 3.0;     // reported norm after such a stop: kFPredictBound * s2
constexpr int kFSweeps = 5;           // fixed-point sweeps of the starting point

struct FastLayout {
    int KP;
    int d, tg, p, r, key, psi, Dr, alpha, alpha_prev, delta, w, g, g2, col, gw, g2w, tq, cq, scal, uni;
    int jacc_bytes_off, ints, total_bytes, uni_doubles;
    __host__ __device__ FastLayout(int KP_, int NT) : KP(KP_) {
        int o = 0;
        d = o; o += KP; tg = o; o += KP; p = o; o += KP; r = o; o += KP; key = o; o += KP;
        psi = o; o += KP + 4; Dr = o; o += KP + 4;
        alpha = o; o += KP; alpha_prev = o; o += KP; delta = o; o += KP; w = o; o += KP; g = o; o += KP;
        g2 = o; o += KP; col = o; o += kMP;
        gw = o; o += kFW * KP; g2w = o; o += kFW * KP;
        tq = o; o += kFMaxNodes; cq = o; o += kFMaxNodes;
        scal = o; o += 48;
        uni = o;
        // union: staging of the Hessian operands (two float arrays [kJC * NT][kMS]) / vectors of the Newton step
        const int stage_doubles = (2 * kJC * NT * kMS * 4 + 7) / 8;
        const int jmat_doubles = 2 * (kMP + 4) + 2 * kMP;    // (floats, so twice what is needed) pivot row / column buffers
        uni_doubles = stage_doubles > jmat_doubles ? stage_doubles : jmat_doubles;
        o += uni_doubles;
        jacc_bytes_off = o * 8;                       // float [kMP][kMP] accumulator of the contraction
        o += (kMP * (kMP + 1) + 1) / 2;
        ints = o * 8;
        total_bytes = ints + KP * 4 * 4 + 64;
    }
};
static inline int fast_smem_bytes(int KP, int NT) { return FastLayout(KP, NT).total_bytes; }

struct FSm {
    GR_PTR(double) d, tg, p, r, key, psi, Dr, alpha, alpha_prev, delta, w, g, g2, col, gw, g2w, tq, cq, scal, J;
    GR_PTR(float) AS, HS, Jacc;
    GR_PTR(int) id, blk, itmp, trunc;
    int KP;
};
enum { SC_Q = 0, SC_FAIL = 1, SC_RED = 8, SC_GRID = 24 };   // (SC_RED: one slot per warp; 16..23: preparation outputs;
                                                            //  SC_GRID: two slots per warp)

__device__ __forceinline__ double ipow(double x, int n) {
    double r = 1.0;
    while (n > 0) { if (n & 1) r *= x; x *= x; n >>= 1; }
    return r;
}

// exp(-y) for y >= 0 (fp64): range reduction by ln 2 and a degree-13 Taylor polynomial on |r| <= ln2/2
// (truncation below 1e-17 relative); results below 2^-1000 are flushed to zero.
__device__ __forceinline__ double exp_neg(double y)
{
    const double t = -y;
    const double kf = rint(t * 1.4426950408889634);
    if (kf < -1000.0) return 0.0;
    double r = fma(-kf, 6.93147180369123816490e-01, t);
    r = fma(-kf, 1.90821492927058770002e-10, r);
    double p = 1.6059043836821613e-10;                 // 1/13!
    p = fma(p, r, 2.08767569878681e-09);               // 1/12!
    p = fma(p, r, 2.505210838544172e-08);              // 1/11!
    p = fma(p, r, 2.755731922398589e-07);              // 1/10!
    p = fma(p, r, 2.7557319223985893e-06);             // 1/9!
    p = fma(p, r, 2.48015873015873e-05);               // 1/8!
    p = fma(p, r, 1.984126984126984e-04);              // 1/7!
    p = fma(p, r, 1.388888888888889e-03);              // 1/6!
    p = fma(p, r, 8.333333333333333e-03);              // 1/5!
    p = fma(p, r, 4.1666666666666664e-02);             // 1/4!
    p = fma(p, r, 1.6666666666666666e-01);             // 1/3!
    p = fma(p, r, 0.5);
    p = fma(p, r, 1.0);
    p = fma(p, r, 1.0);
    const int k = (int)kf;
    return __hiloint2double(__double2hiint(p) + (k << 20), __double2loint(p));
}

__device__ __forceinline__ constexpr double inv_fact(int c) {
    double f = 1.0;
    for (int i = 2; i <= c; i++) f *= (double)i;
    return 1.0 / f;
}

// hh[c], c = 1..NT: coefficients of (e^mu - 1) / (1 + x (e^mu - 1)) in mu.  Column-oriented so that the
// dependent chain is two operations per coefficient.
template <int NT>
__device__ __forceinline__ void unit_h_series(double x, double* hh)
{
    double acc[NT + 1];
#pragma unroll
    for (int c = 1; c <= NT; c++) acc[c] = 0.0;
    hh[1] = 1.0;
#pragma unroll
    for (int k = 1; k < NT; k++) {
#pragma unroll
        for (int c = k + 1; c <= NT; c++) acc[c] = fma(inv_fact(c - k), hh[k], acc[c]);
        hh[k + 1] = fma(-x, acc[k + 1], inv_fact(k + 1));
    }
}

__device__ __forceinline__ double warp_sum_d(double v) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum of NT-entry vectors over the 32 lanes, result in every lane.  Recursive halving: at each of the
// first log2(NT) levels a lane keeps half of its entries and hands the other half to its partner, so the
// exchange costs NT - 1 + (5 - log2 NT) shuffles instead of 5 NT; an all-gather of NT shuffles follows.
template <int NT>
__device__ __forceinline__ void warp_allreduce_series(double* S, int lane)
{
    static_assert(NT == 4 || NT == 8 || NT == 16, "series length");
    int cnt = NT, o = 16;
#pragma unroll
    for (int lvl = 0; lvl < (NT == 16 ? 4 : (NT == 8 ? 3 : 2)); lvl++) {
        const int half = cnt >> 1;
        const bool up = (lane & o) != 0;
#pragma unroll
        for (int c = 0; c < NT / 2; c++) {
            if (c < half) {
                const double keep = up ? S[c + half] : S[c];
                const double send = up ? S[c] : S[c + half];
                S[c] = keep + __shfl_xor_sync(0xffffffffu, send, o);
            }
        }
        cnt = half; o >>= 1;
    }
    double v = S[0];
    for (; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    // lane bits (4, 3[, 2[, 1]]) say which entry the lane holds
#pragma unroll
    for (int c = 0; c < NT; c++) {
        const int src = (NT == 16) ? ((((c >> 3) & 1) << 4) | (((c >> 2) & 1) << 3) | (((c >> 1) & 1) << 2) | ((c & 1) << 1))
                      : (NT == 8) ? ((((c >> 2) & 1) << 4) | (((c >> 1) & 1) << 3) | ((c & 1) << 2))
                                  : ((((c >> 1) & 1) << 4) | ((c & 1) << 3));
        S[c] = __shfl_sync(0xffffffffu, v, src);
    }
}

// tf32 rounding of a staged operand (the contraction runs on the tensor cores: it is the one dense
// contraction of the path, and it only steers Newton's method)
__device__ __forceinline__ float to_tf32(float x) {
    uint32_t u;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(x));
    return __uint_as_float(u);
}

// Series of length 16 cancel too strongly for one tf32 product (a dominant draft token makes the terms of
// sum_kappa A[n - kappa] h[kappa] alternate at ~1e3 times their sum): their operands are staged in full fp32 and
// split into two tf32 parts when the fragments are loaded (three MMAs per tile step, error ~1e-6 per term).
template <int NT>
__device__ __forceinline__ float stage_round(float x) { return NT > 8 ? x : to_tf32(x); }

__device__ __forceinline__ void mma_tf32(float& c0, float& c1, float& c2, float& c3, uint32_t a0, uint32_t a1,
                                         uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c0), "+f"(c1), "+f"(c2), "+f"(c3)
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// One chunk of the Hessian contraction: Jacc[i][l] += sum over the staged rows kk of AS[kk][i] HS[kk][l] for the
// 16 x 8 tiles that touch the lower triangle, as m16n8k8 tf32 MMAs with fp32 accumulation.  K8 = staged rows,
// a multiple of 8.  The lower tiles are dealt round-robin to the warps.
template <bool kSplit>
__device__ __forceinline__ void hess_chunk(const FSm& sm, int K8, int m)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gid = lane >> 2, tig = lane & 3;
    // tile (mi, ni), ni <= 2 mi + 1, has the running number mi (mi + 1) + ni
    for (int t = warp; t < (kMP / 16) * (kMP / 16 + 1); t += kFW) {
        int mi = 0;
        while ((mi + 1) * (mi + 2) <= t) mi++;
        const int ni = t - mi * (mi + 1);
        const int i0 = 16 * mi, l0 = 8 * ni;
        if (i0 >= m || l0 >= m) continue;
        float c0 = 0.f, c1 = 0.f, c2 = 0.f, c3 = 0.f;
        for (int k0 = 0; k0 < K8; k0 += 8) {
            GR_PTR(const float) Ap = sm.AS + ((k0 + tig) * kMS + i0 + gid);
            GR_PTR(const float) Bp = sm.HS + ((k0 + tig) * kMS + l0 + gid);
            const float fa[4] = {Ap[0], Ap[8], Ap[4 * kMS], Ap[4 * kMS + 8]};
            const float fb[2] = {Bp[0], Bp[4 * kMS]};
            if (kSplit) {
                uint32_t ah[4], al[4], bh[2], bl[2];
#pragma unroll
                for (int z = 0; z < 4; z++) {
                    const float hi = to_tf32(fa[z]);
                    ah[z] = __float_as_uint(hi); al[z] = __float_as_uint(to_tf32(fa[z] - hi));
                }
#pragma unroll
                for (int z = 0; z < 2; z++) {
                    const float hi = to_tf32(fb[z]);
                    bh[z] = __float_as_uint(hi); bl[z] = __float_as_uint(to_tf32(fb[z] - hi));
                }
                mma_tf32(c0, c1, c2, c3, al[0], al[1], al[2], al[3], bh[0], bh[1]);
                mma_tf32(c0, c1, c2, c3, ah[0], ah[1], ah[2], ah[3], bl[0], bl[1]);
                mma_tf32(c0, c1, c2, c3, ah[0], ah[1], ah[2], ah[3], bh[0], bh[1]);
            } else {
                mma_tf32(c0, c1, c2, c3, __float_as_uint(fa[0]), __float_as_uint(fa[1]), __float_as_uint(fa[2]),
                         __float_as_uint(fa[3]), __float_as_uint(fb[0]), __float_as_uint(fb[1]));
            }
        }
        GR_PTR(float) J0 = sm.Jacc + ((i0 + gid) * kJS + l0 + 2 * tig);
        J0[0] += c0; J0[1] += c1;
        J0[8 * kJS] += c2; J0[8 * kJS + 1] += c3;
    }
}

// g (always), and with want_jac the diagonal part g2 and the contraction Jacc, at the weights in sm.w.
// The contraction takes every jstride-th node (weights scaled by jstride).
// Node abscissae / weights are in sm.tq / sm.cq, their number in sm.scal[SC_Q].
template <int NT, int TPL>
__device__ void fast_eval(const FSm& sm, int m, int n, GR_PTR(const double) d, double hmass, bool want_jac, int jstride)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, KP = sm.KP;
    const int Q = (int)sm.scal[SC_Q];
    double wr[TPL], dr[TPL], gacc[TPL], g2acc[TPL];
#pragma unroll
    for (int tt = 0; tt < TPL; tt++) {
        const int j = lane + 32 * tt;
        wr[tt] = j < m ? sm.w[j] : 0.0;
        dr[tt] = j < m ? d[j] : 0.0;
        gacc[tt] = 0.0; g2acc[tt] = 0.0;
    }
    if (want_jac) {
        for (int e = tid; e < kMP * kJS; e += kFT) sm.Jacc[e] = 0.f;
    }
    const int span = jstride * kJC;      // nodes per chunk: every jstride-th one is a Hessian node
    for (int q0 = 0; q0 < Q; q0 += span) {
        const int q1 = min(Q, q0 + span);
        for (int q = q0 + warp; q < q1; q += kFW) {
            const double t = sm.tq[q];
            double S[NT];
#pragma unroll
            for (int c = 0; c < NT; c++) S[c] = 0.0;
            double xk[TPL];
#pragma unroll
            for (int tt = 0; tt < TPL; tt++) {
                const double x = exp_neg(t * wr[tt]);
                xk[tt] = x;
                double hh[NT + 1];
                unit_h_series<NT>(x, hh);
                // h[c] = d^c hh[c];  S[0] += x d,  S[c] += x (1 - x) d h[c]
                const double dd = dr[tt];
                S[0] = fma(x, dd, S[0]);
                double pw = x * (1.0 - x) * dd;
#pragma unroll
                for (int c = 1; c < NT; c++) {
                    pw *= dd;
                    S[c] = fma(pw, hh[c], S[c]);
                }
            }
            // log-derivative of the product: sum over the tokens (all lanes end with the totals)
            warp_allreduce_series<NT>(S, lane);
            S[0] += hmass;
            // P' = S P, column-oriented
            double P[NT + 1], acc[NT + 1];
            P[0] = 1.0;
#pragma unroll
            for (int c = 1; c <= NT; c++) acc[c] = 0.0;
#pragma unroll
            for (int k = 0; k < NT; k++) {
#pragma unroll
                for (int c = k + 1; c <= NT; c++) acc[c] = fma(S[c - 1 - k], P[k], acc[c]);
                P[k + 1] = acc[k + 1] * (1.0 / (double)(k + 1));
            }
            // R[c] = P[n - c]: the coefficient that pairs with h[c] in [lambda^n] P h
            // (for n < NT: the reversed series moved down by NT - n places, one conditional move per bit)
            double R[NT + 1];
#pragma unroll
            for (int c = 1; c <= NT; c++) R[c] = P[NT - c];
            if (n != NT) {
                const int sh = NT - n;
#pragma unroll
                for (int bit = NT / 2; bit >= 1; bit >>= 1) {
                    if (sh & bit) {
#pragma unroll
                        for (int c = 1; c <= NT; c++) R[c] = (c + bit <= NT) ? R[c + bit] : 0.0;
                    }
                }
            }
            const double cq = sm.cq[q];
            const bool jnode = want_jac && ((q - q0) % jstride == 0);
            const int slot = (q - q0) / jstride;
#pragma unroll
            for (int tt = 0; tt < TPL; tt++) {
                double hh[NT + 1], hd[NT + 1];
                unit_h_series<NT>(xk[tt], hh);
                const double dd = dr[tt];
                double pw = 1.0, val = 0.0;
#pragma unroll
                for (int c = 1; c <= NT; c++) {
                    pw *= dd;
                    hd[c] = pw * hh[c];                 // h[c] = d^c hh[c]
                    val = fma(R[c], hd[c], val);
                }
                const double u = wr[tt] * xk[tt];
                const double gi = cq * u * val;
                gacc[tt] += gi;
                g2acc[tt] = fma(gi * t, wr[tt], g2acc[tt]);
                if (jnode) {
                    // A = P h (series), paired as  sum_kappa A[n - kappa] h_l[kappa],  kappa = 1..n-1.
                    // Staged scaled: AS = 2 c_q t u A[n - kappa] (the 2: every second node), HS = u h[kappa].
                    // Row kappa - 1 of the node's slot holds the pair (A[n - kappa], h[kappa]); rows n - 1 .. NT - 1
                    // are zero (they pad the contraction length to a multiple of the MMA depth).
                    const int j = lane + 32 * tt;
                    const double sa = (double)jstride * cq * t * u;
                    GR_PTR(float) as = sm.AS + (slot * NT * kMS + j);
                    GR_PTR(float) hs = sm.HS + (slot * NT * kMS + j);
                    if (n == NT) {
                        // full series length: fixed rows, each A consumed as soon as it is formed
#pragma unroll
                        for (int kap = 1; kap < NT; kap++) {
                            double a = 0.0;              // A[NT - kap] = sum_c h[c] P[NT - kap - c]
#pragma unroll
                            for (int c = 1; c <= NT - kap; c++) a = fma(hd[c], P[NT - kap - c], a);
                            as[(kap - 1) * kMS] = stage_round<NT>((float)(sa * a));
                            hs[(kap - 1) * kMS] = stage_round<NT>((float)(u * hd[kap]));
                            if (TPL == 1) { as[(kap - 1) * kMS + 32] = 0.f; hs[(kap - 1) * kMS + 32] = 0.f; }
                        }
                        as[(NT - 1) * kMS] = 0.f; hs[(NT - 1) * kMS] = 0.f;
                        if (TPL == 1) { as[(NT - 1) * kMS + 32] = 0.f; hs[(NT - 1) * kMS + 32] = 0.f; }
                    } else {
#pragma unroll
                        for (int e2 = 1; e2 < NT; e2++) {
                            double a = 0.0;              // A[e2] = sum_{c=1..e2} h[c] P[e2 - c]
#pragma unroll
                            for (int c = 1; c <= e2; c++) a = fma(hd[c], P[e2 - c], a);
                            if (e2 < n) as[(n - e2 - 1) * kMS] = stage_round<NT>((float)(sa * a));
                        }
#pragma unroll
                        for (int kap = 1; kap <= NT; kap++) {
                            const bool live = kap < n;
                            if (!live) as[(kap - 1) * kMS] = 0.f;
                            hs[(kap - 1) * kMS] = live ? stage_round<NT>((float)(u * hd[kap])) : 0.f;
                            if (TPL == 1) { as[(kap - 1) * kMS + 32] = 0.f; hs[(kap - 1) * kMS + 32] = 0.f; }
                        }
                    }
                }
            }
        }
        if (want_jac) {
            const int nstaged = (q1 - q0 + jstride - 1) / jstride;
            int K8 = nstaged * NT;
            if (K8 & 7) {
                // NT = 4 with an odd number of staged nodes: one more all-zero slot completes the MMA depth
                for (int e = tid; e < NT * kMS; e += kFT) { sm.AS[K8 * kMS + e] = 0.f; sm.HS[K8 * kMS + e] = 0.f; }
                K8 += NT;
            }
            __syncthreads();
            hess_chunk<(NT > 8)>(sm, K8, m);
            __syncthreads();
        }
    }
#pragma unroll
    for (int tt = 0; tt < TPL; tt++) {
        const int j = lane + 32 * tt;
        if (j < m) { sm.gw[warp * KP + j] = gacc[tt]; sm.g2w[warp * KP + j] = g2acc[tt]; }
    }
    __syncthreads();
    if (tid < m) {
        double a = 0.0, b2 = 0.0;
#pragma unroll
        for (int w2 = 0; w2 < kFW; w2++) { a += sm.gw[w2 * KP + tid]; b2 += sm.g2w[w2 * KP + tid]; }
        sm.g[tid] = a; sm.g2[tid] = b2;
    }
    __syncthreads();
}

// w = exp(alpha), its range, and the quadrature grid for it.
static __device__ void fast_grid(const FSm& sm, int m, int n, int slack, double qstep)
{
    const int tid = threadIdx.x;
    GR_PTR(double) red = sm.scal + SC_GRID;
    double a = 0.0;
    if (tid < m) { a = sm.alpha[tid]; sm.w[tid] = exp(a); }
    // extreme alphas in one pass (they give the extreme weights)
    double hi = tid < m ? a : -1.0e300, lo = tid < m ? -a : -1.0e300;
    for (int o = 16; o > 0; o >>= 1) {
        hi = fmax(hi, __shfl_xor_sync(0xffffffffu, hi, o));
        lo = fmax(lo, __shfl_xor_sync(0xffffffffu, lo, o));
    }
    __syncthreads();
    if ((tid & 31) == 0) { red[2 * (tid >> 5)] = hi; red[2 * (tid >> 5) + 1] = lo; }
    __syncthreads();
    hi = red[0]; lo = red[1];
#pragma unroll
    for (int i = 1; i < kFW; i++) { hi = fmax(hi, red[2 * i]); lo = fmax(lo, red[2 * i + 1]); }
    lo = -lo;
    const double wmax = exp(hi), wmin = exp(lo);
    const double rate = slack ? 1.0 + wmin : wmin;
    const double s_hi = log(kFTEnd / rate);
    const double s0 = -log((slack ? 1.0 : 0.0) + wmax) - kFDrop;
    int Q = (int)ceil((s_hi - (s0 - kFTail)) / qstep) + 1;
    if (Q > kFMaxNodes) Q = kFMaxNodes;
    double nfact = 1.0;
    for (int c = 2; c <= n; c++) nfact *= (double)c;
    for (int q = tid; q < Q; q += kFT) {
        const double s = s_hi - qstep * (double)q;
        const double e = exp(-(s - s0));
        const double t = exp(s - e);
        sm.tq[q] = t;
        sm.cq[q] = qstep * (1.0 + e) * t * (slack ? exp(-t) : 1.0) * nfact;
    }
    if (tid == 0) sm.scal[SC_Q] = (double)Q;
    __syncthreads();
}

// Newton step: fp32 Cholesky of the Hessian in place in the contraction accumulator (row stride kJS),
// with the forward substitution carried along and the backward substitution on warp 0.  The step only
// steers the iteration (the fp64 gradient decides convergence) and the Hessian was accumulated in fp32.
// Matrix: off-diagonal -Jacc (lower triangle), diagonal g - g2, plus `add` everywhere.  Writes the step
// into sm.delta; sets SC_FAIL when a pivot is not positive.
static __device__ void fast_newton_step(const FSm& sm, int m, GR_PTR(const double) rhs, double add)
{
    const int tid = threadIdx.x;
    GR_PTR(float) Jm = sm.Jacc;
    GR_PTR(float) yv = GR_PCAST(float, sm.J);          // [kMP] working right-hand side
    GR_PTR(float) yf = yv + kMP;                       // [kMP] forward-substituted right-hand side, then the solution
    GR_PTR(float) dg = yf + kMP;                       // [kMP] diagonal of the factor
    const float addf = (float)add;
    for (int e = tid; e < m * kMP; e += kFT) {
        const int i = e / kMP, l = e & (kMP - 1);
        if (l < i) Jm[i * kJS + l] = addf - Jm[i * kJS + l];
    }
    if (tid < m) {
        Jm[tid * kJS + tid] = (float)(sm.g[tid] - sm.g2[tid]) + addf;
        // Right-hand side.  Along its own coordinate a token's flow behaves like a logistic curve
        // g_i = c sigma(alpha_i - kappa): linear in w_i while the token is light, saturating at the flow c of the
        // tuples it can win at all once it is heavy.  The curve through the current value and slope
        // (H_ii = g_i (1 - g_i / c)  gives  c = g_i^2 / g2_i)  is inverted exactly:  H_ii (logit(rhs_i / c) -
        // logit(g_i / c))  replaces  rhs_i - g_i.  Near the solution the two agree to first order; far from it a
        // token close to saturation (weight in the thousands) is placed at once, where the plain residual moves
        // its weight by a factor e per step, and a light token gets the multiplicative update log(rhs_i / g_i).
        const double gi = sm.g[tid], g2i = sm.g2[tid], ri = rhs[tid];
        // (a target at or beyond the saturation level this curve predicts says that the curve is off: the plain
        // residual is used for that token; without this a single token of weight ~1e5 crawled for 40 steps)
        const double room = 1.0 - ri * g2i / (gi * gi);
        const double arg = fmax((ri - gi) / (gi * fmax(room, 1e-3)), -1.0 + 1e-12);
        yv[tid] = (float)(room > 1e-3 ? (gi - g2i) * log1p(arg) : ri - gi);
    }
    __syncthreads();
    bool bad = false;
    // Blocked right-looking factorisation in panels of eight columns: every thread factors the 8 x 8 diagonal block
    // in registers (redundantly: no exchange needed), one thread per row solves the panel below it and carries the
    // forward substitution along, and the rest of the matrix takes the panel's rank-8 update on the tensor cores.
    for (int j0 = 0; j0 < m; j0 += 8) {
        const int nb = min(8, m - j0);
        float Lb[8][8], yb[8], dinv[8];
#pragma unroll
        for (int c = 0; c < 8; c++) {
#pragma unroll
            for (int c2 = 0; c2 <= c; c2++) Lb[c][c2] = (c < nb) ? Jm[(j0 + c) * kJS + j0 + c2] : (c == c2 ? 1.f : 0.f);
            yb[c] = (c < nb) ? yv[j0 + c] : 0.f;
        }
#pragma unroll
        for (int c = 0; c < 8; c++) {
            const float dv = Lb[c][c];
            if (!(dv > 0.f)) bad = true;
            dinv[c] = rsqrtf(dv);
            Lb[c][c] = dv * dinv[c];
            yb[c] *= dinv[c];
#pragma unroll
            for (int r2 = c + 1; r2 < 8; r2++) Lb[r2][c] *= dinv[c];
#pragma unroll
            for (int r2 = c + 1; r2 < 8; r2++) {
#pragma unroll
                for (int c3 = c + 1; c3 <= r2; c3++) Lb[r2][c3] = fmaf(-Lb[r2][c], Lb[c3][c], Lb[r2][c3]);
                yb[r2] = fmaf(-Lb[r2][c], yb[c], yb[r2]);
            }
        }
        if (bad) break;
        // panel below the block: one row per thread (it touches no entry of the block itself)
        const int i1 = j0 + nb + tid;
        if (i1 < m) {
            float v[8];
#pragma unroll
            for (int c = 0; c < 8; c++) v[c] = (c < nb) ? Jm[i1 * kJS + j0 + c] : 0.f;
            float yi = yv[i1];
#pragma unroll
            for (int c = 0; c < 8; c++) {
                const float lc = v[c] * dinv[c];
#pragma unroll
                for (int c3 = c + 1; c3 < 8; c3++) v[c3] = fmaf(-lc, Lb[c3][c], v[c3]);
                yi = fmaf(-lc, yb[c], yi);
                if (c < nb) Jm[i1 * kJS + j0 + c] = lc;
            }
            yv[i1] = yi;
        }
        __syncthreads();
        // every thread has read the block by now: one of them stores its factor
        if (tid == kFT - 1) {
#pragma unroll
            for (int c = 0; c < 8; c++) {
                if (c < nb) {
                    dg[j0 + c] = Lb[c][c]; yf[j0 + c] = yb[c];
#pragma unroll
                    for (int c2 = 0; c2 < c; c2++) Jm[(j0 + c) * kJS + j0 + c2] = Lb[c][c2];
                }
            }
        }
        // trailing update  J[i][l] -= sum_c L[i][c] L[l][c],  j0 + 8 <= l <= i:  m16n8k8 MMAs on the 16 x 8 tiles of
        // the lower triangle, operands split into two tf32 parts (~fp32 products)
        const int t0 = j0 + 8;
        if (t0 < m) {
            const int lane = tid & 31, warp = tid >> 5, gid = lane >> 2, tig = lane & 3;
            // tile t of the lower triangle: row mi of 16-row tiles holds tiles mi (mi + 1) .. (mi + 1)(mi + 2) - 1
            // (2 mi + 2 of them); each warp takes every kFW-th tile and finds (mi, ni) from t directly
            const int nmt = (m - t0 + 15) >> 4;
            for (int t = warp; t < nmt * (nmt + 1); t += kFW) {
                int mi = (int)((sqrtf((float)(4 * t + 1)) - 1.f) * 0.5f);
                while (mi * (mi + 1) > t) mi--;
                while ((mi + 1) * (mi + 2) <= t) mi++;
                const int ni = t - mi * (mi + 1);
                {
                    if (t0 + 8 * ni >= m) continue;
                    const int ra = t0 + 16 * mi + gid, rb = ra + 8, l0 = t0 + 8 * ni, cb = l0 + gid;
                    const bool oa = ra < m, ob = rb < m, oc = cb < m;
                    const float fa[4] = {oa ? -Jm[ra * kJS + j0 + tig] : 0.f, ob ? -Jm[rb * kJS + j0 + tig] : 0.f,
                                         oa ? -Jm[ra * kJS + j0 + tig + 4] : 0.f, ob ? -Jm[rb * kJS + j0 + tig + 4] : 0.f};
                    const float fb[2] = {oc ? Jm[cb * kJS + j0 + tig] : 0.f, oc ? Jm[cb * kJS + j0 + tig + 4] : 0.f};
                    GR_PTR(float) C0 = Jm + (ra * kJS + l0 + 2 * tig);
                    GR_PTR(float) C1 = Jm + (rb * kJS + l0 + 2 * tig);
                    float c0 = oa ? C0[0] : 0.f, c1 = oa ? C0[1] : 0.f, c2 = ob ? C1[0] : 0.f, c3 = ob ? C1[1] : 0.f;
                    uint32_t ah[4], al[4], bh[2], bl[2];
#pragma unroll
                    for (int z = 0; z < 4; z++) {
                        const float hi = to_tf32(fa[z]);
                        ah[z] = __float_as_uint(hi); al[z] = __float_as_uint(to_tf32(fa[z] - hi));
                    }
#pragma unroll
                    for (int z = 0; z < 2; z++) {
                        const float hi = to_tf32(fb[z]);
                        bh[z] = __float_as_uint(hi); bl[z] = __float_as_uint(to_tf32(fb[z] - hi));
                    }
                    // three independent accumulations (the small cross terms apart), summed afterwards
                    float e0 = 0.f, e1 = 0.f, e2 = 0.f, e3 = 0.f, f0 = 0.f, f1 = 0.f, f2 = 0.f, f3 = 0.f;
                    mma_tf32(e0, e1, e2, e3, al[0], al[1], al[2], al[3], bh[0], bh[1]);
                    mma_tf32(f0, f1, f2, f3, ah[0], ah[1], ah[2], ah[3], bl[0], bl[1]);
                    mma_tf32(c0, c1, c2, c3, ah[0], ah[1], ah[2], ah[3], bh[0], bh[1]);
                    if (oa) { C0[0] = c0 + (e0 + f0); C0[1] = c1 + (e1 + f1); }
                    if (ob) { C1[0] = c2 + (e2 + f2); C1[1] = c3 + (e3 + f3); }
                }
            }
        }
        __syncthreads();
    }
    if (bad) {
        if (tid == 0) sm.scal[SC_FAIL] = 1.0;
        __syncthreads();
        return;
    }
    // backward substitution L^T x = y on warp 0, column-oriented with the right-hand side in registers (lane l holds
    // entries l, l + 32, ...): unknown e is finished by its owner, broadcast, and taken out of the entries above it.
    // One multiply, one shuffle and one FMA per unknown on the critical path; row e of L is fetched one step ahead.
    if (tid < 32 && kRL == 2) {
        // (two entries per lane, written out: the general form below compiles to slower code for them)
        const int lane = tid;
        float y0 = lane < m ? yf[lane] : 0.f, y1 = lane + 32 < m ? yf[lane + 32] : 0.f;
        const float r0 = lane < m ? 1.f / dg[lane] : 0.f, r1 = lane + 32 < m ? 1.f / dg[lane + 32] : 0.f;
        float a0n = Jm[(m - 1) * kJS + lane], a1n = Jm[(m - 1) * kJS + lane + 32];
        for (int e = m - 1; e >= 0; e--) {
            const float a0 = a0n, a1 = a1n;
            if (e > 0) { a0n = Jm[(e - 1) * kJS + lane]; a1n = Jm[(e - 1) * kJS + lane + 32]; }
            const float xe = __shfl_sync(0xffffffffu, (e & 32) ? y1 * r1 : y0 * r0, e & 31);
            if (lane == (e & 31)) {
                if (e & 32) y1 = xe; else y0 = xe;
            }
            if (lane < e) y0 = fmaf(-a0, xe, y0);
            if (lane + 32 < e) y1 = fmaf(-a1, xe, y1);
        }
        if (lane < m) yf[lane] = y0;
        if (lane + 32 < m) yf[lane + 32] = y1;
    }
    if (kRL != 2) {
        // Wider supports: blocked, eight unknowns at a time from the last panel down.  Every thread keeps its own entry
        // of the right-hand side in a register; the block's eight entries go through shared memory (two buffers in
        // turn, one barrier per block), every thread solves the 8 x 8 triangle redundantly and takes the block's
        // unknowns out of its own entry.  About 350 cycles per block, where the one-warp form above spent over 400
        // per unknown at four entries per lane.
        float yl = tid < m ? yf[tid] : 0.f;
        int buf = 0;
        for (int j0 = ((m - 1) >> 3) << 3; j0 >= 0; j0 -= 8) {
            const int nb = min(8, m - j0);
            GR_PTR(float) yb = yv + 8 * buf;
            if (tid >= j0 && tid < j0 + nb) yb[tid - j0] = yl;
            __syncthreads();
            float x[8];
#pragma unroll
            for (int c = 7; c >= 0; c--) {
                float v = 0.f;
                if (c < nb) {
                    v = yb[c];
#pragma unroll
                    for (int c2 = 7; c2 > c; c2--)
                        if (c2 < nb) v = fmaf(-Jm[(j0 + c2) * kJS + j0 + c], x[c2], v);
                    v = v / dg[j0 + c];
                }
                x[c] = v;
            }
            if (tid < j0) {
#pragma unroll
                for (int c = 0; c < 8; c++)
                    if (c < nb) yl = fmaf(-Jm[(j0 + c) * kJS + tid], x[c], yl);
            }
            if (tid == kFT - 1) {
#pragma unroll
                for (int c = 0; c < 8; c++)
                    if (c < nb) yf[j0 + c] = x[c];
            }
            buf ^= 1;
        }
    }
    __syncthreads();
    if (tid < m) sm.delta[tid] = (double)yf[tid];
    __syncthreads();
}

// Smallest pivot of the last factorisation relative to the diagonal entry it came from: how much of the diagonal the
// elimination left (near 1 for a well-conditioned system; 1e-3 and below where the fp32 system is close to singular
// and its solution no longer a Newton step).  Reads the factor's diagonal where fast_newton_step left it.
static __device__ double fast_relative_pivot(const FSm& sm, int m, double add)
{
    const int tid = threadIdx.x;
    GR_PTR(float) dg = GR_PCAST(float, sm.J) + 2 * kMP;
    const double rp = tid < m ? (double)dg[tid] * (double)dg[tid] / (sm.g[tid] - sm.g2[tid] + add) : 1.0;
    return -block_reduce_max(-rp, sm.scal + SC_RED);
}

// Newton iteration for one system.  On return sm.w holds exp(alpha) at the last evaluated point.
template <int NT, int TPL>
__device__ int fast_system(const FSm& sm, int m, int n, GR_PTR(const double) d, GR_PTR(const double) rhs, double hmass,
                           int slack, double tol, int max_iters, double qstep, double* gnorm, int* iters)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    GR_PTR(double) red = sm.scal + SC_RED;
    // ---- mean-field starting point: token i wins the share w_i / (slack + w_i + S_i) of the tuples that
    //      contain it, S_i = expected weight of the other drafted tokens given that i was drafted
    const double T = hmass + block_reduce_sum(tid < m ? d[tid] : 0.0, red);
    const double Tn = ipow(T, n);
    double ci = 1.0, rho = 0.5, wi = 1.0;
    if (tid < m) {
        sm.col[tid] = ipow(fmax(T - d[tid], 0.0), n);        // mass of tuples avoiding token tid
        ci = Tn - sm.col[tid];
        rho = fmin(rhs[tid] / ci, 1.0 - 1e-3);
        wi = slack ? rho / (1.0 - rho) : rhs[tid] / d[tid];
    }
    if (!slack) {
        const double ml = block_reduce_sum(tid < m ? log(wi) : 0.0, red) / (double)m;
        wi *= exp(-ml);
    }
    if (tid < m) sm.w[tid] = wi;
    __syncthreads();
    // Pr[i and j drafted, all drafts inside] once, in the (still unused) contraction accumulator
    for (int e = tid; e < m * kMP; e += kFT) {
        const int i = e / kMP, j = e - i * kMP;
        if (j < m) {
            const double pij = Tn - sm.col[i] - sm.col[j] + ipow(fmax(T - d[i] - d[j], 0.0), n);
            sm.Jacc[i * kJS + j] = (i == j) ? 0.f : (float)pij;
        }
    }
    __syncthreads();
    // Sweeps of  w_i = rho_i / (1 - rho_i) * (slack + S_i),  S_i = the weight token i is up against.  A competitor j,
    // present with probability pi_ij = Pr[i and j drafted] / Pr[i drafted], adds to S_i the weight e_j for which
    // 1 / (A + e_j) = (1 - pi_ij) / A + pi_ij / (A + w_j),  A = slack + w_i + S_i:  e_j = A pi_ij w_j / (A + w_j (1 - pi_ij)).
    // For w_j << A this is the mean-field value pi_ij w_j; a huge w_j counts for A pi_ij / (1 - pi_ij) only (token i
    // simply loses the tuples that contain j), which keeps the start sane when a few weights are in the thousands.
    // fp32: it is a starting point.
    if (tid < m) { sm.g2[tid] = 1.0 / ci; sm.g[tid] = (slack ? 1.0 : 0.0) + wi; }
    __syncthreads();
    GR_PTR(float) part = sm.AS;                       // [kFW][kMP] partial sums (the staging area is idle here)
    for (int sweep = 0; sweep < kFSweeps; sweep++) {
        // lane = rows lane, lane + 32, ...; warp = a contiguous share of the columns: no shuffles, independent sums
        {
            const int chunk = (m + kFW - 1) / kFW;
            const int jlo = warp * chunk, jhi = min(m, jlo + chunk);
            float Ar[kRL], cr[kRL], sa[kRL], sb[kRL];
            GR_PTR(const float) row[kRL];
#pragma unroll
            for (int u = 0; u < kRL; u++) {
                const int r = lane + 32 * u;
                const bool on = r < m;
                Ar[u] = on ? (float)sm.g[r] : 1.f; cr[u] = on ? (float)sm.g2[r] : 0.f;
                row[u] = sm.Jacc + ((on ? r : 0) * kJS);
                sa[u] = 0.f; sb[u] = 0.f;
            }
            int j = jlo;
            for (; j + 1 < jhi; j += 2) {
                const float wa = (float)sm.w[j], wb = (float)sm.w[j + 1];
#pragma unroll
                for (int u = 0; u < kRL; u++) {
                    const float pa = fminf(row[u][j] * cr[u], 1.f), pb = fminf(row[u][j + 1] * cr[u], 1.f);
                    sa[u] += __fdividef(Ar[u] * pa * wa, Ar[u] + wa * (1.f - pa));
                    sb[u] += __fdividef(Ar[u] * pb * wb, Ar[u] + wb * (1.f - pb));
                }
            }
            if (j < jhi) {
                const float wa = (float)sm.w[j];
#pragma unroll
                for (int u = 0; u < kRL; u++) {
                    const float pa = fminf(row[u][j] * cr[u], 1.f);
                    sa[u] += __fdividef(Ar[u] * pa * wa, Ar[u] + wa * (1.f - pa));
                }
            }
#pragma unroll
            for (int u = 0; u < kRL; u++) part[warp * kMP + lane + 32 * u] = sa[u] + sb[u];
        }
        __syncthreads();
        double Si = 0.0;
        if (tid < m) {
#pragma unroll
            for (int w2 = 0; w2 < kFW; w2++) Si += (double)part[w2 * kMP + tid];
            wi = rho / (1.0 - rho) * (slack ? 1.0 + Si : fmax(Si, 1e-300));
        }
        double scale = 1.0;
        if (!slack) {
            const double ml = block_reduce_sum(tid < m ? log(wi) : 0.0, red) / (double)m;
            scale = exp(-ml);
            wi *= scale;
        }
        __syncthreads();
        if (tid < m) { sm.w[tid] = wi; sm.g[tid] = (slack ? 1.0 : 0.0) + wi + scale * Si; }
        __syncthreads();
    }
    if (tid < m) {
        sm.alpha[tid] = fmin(fmax(log(wi), -kFAlphaClamp), kFAlphaClamp);
    }
    __syncthreads();

    int status = GR_NOT_CONVERGED, it = 0;
    double rn = 0.0, rprev = 1.0e300, lam = 1.0;
    bool was_coarse = true;
    bool full_grid_only = false;         // set once a factorisation has failed
    int stalls = 0;
    bool predicted = false;              // the norm returned is a prediction, not an evaluation                      // times a step could not be made to reduce the residual at any length tried
    for (; it < max_iters; it++) {
        // far from the solution the trapezoid step is doubled (quadrature error ~4e-6, far below the gradient
        // norm there): half the nodes, every one of them a Hessian node.  Convergence is only ever declared on
        // the full grid.
        const bool coarse = rprev > 1.0e-2 && !full_grid_only;
        fast_grid(sm, m, n, slack, coarse ? 2.0 * qstep : qstep);
        // Hessian nodes: every second one on the full grid, every one on the doubled step (taking every second one
        // there too kept all eight warps of the wide kernel busy and saved 8 % on one shape, but a Hessian from six or
        // seven nodes cost others one to three more evaluations, and a 128-token, n = 16 shape seven times its time)
        fast_eval<NT, TPL>(sm, m, n, d, hmass, true, coarse ? 1 : 2);
        rn = block_reduce_sum(tid < m ? fabs(sm.g[tid] - rhs[tid]) : 0.0, red);
        if (rn <= tol && !coarse) { status = GR_OK; it++; break; }
        // (a residual on the full grid is not compared with the coarse grid's: they differ by the coarse quadrature error)
        const bool comparable = coarse == was_coarse;
        was_coarse = coarse;
        if (comparable && !(rn < rprev) && lam > 1.0 / 64.0 && it > 0) {
            // the last step did not reduce the gradient norm: retry it at half length
            lam *= 0.5;
            if (tid < m) sm.alpha[tid] = sm.alpha_prev[tid] + lam * sm.delta[tid];
            __syncthreads();
            continue;
        }
        // A step that did not reduce the residual even at 1/64 of its length: the fp32 Newton system has reached its
        // accuracy for this instance (weights of 1e5 and more).  The second time the instance is handed to the fp64
        // kernel, which starts from the last accepted point, instead of spending the rest of the evaluation budget.
        if (comparable && !(rn < rprev) && it > 0 && ++stalls >= 2) {
            if (tid < m) sm.alpha[tid] = sm.alpha_prev[tid];
            __syncthreads();
            break;
        }
        // contraction of the last full step (same grid on both sides)
        const double rho = (comparable && !coarse && it > 0 && lam == 1.0) ? rn / rprev : 1.0e300;
        rprev = rn; lam = 1.0;
        if (tid < m) sm.alpha_prev[tid] = sm.alpha[tid];
        if (tid == 0) sm.scal[SC_FAIL] = 0.0;
        // Newton step with the Hessian (off-diagonal from the contraction, diagonal g - g2); an outer block's
        // function is constant along (1,...,1): pin that direction with 1/m everywhere
        fast_newton_step(sm, m, rhs, slack ? 0.0 : 1.0 / (double)m);
        const bool fail = sm.scal[SC_FAIL] != 0.0;
        // (a Hessian from the doubled step that is not positive definite in fp32: with the full grid's diagonal the
        // factorisation usually goes through, where proportional fitting would crawl down to the switch at 1e-2)
        if (fail) full_grid_only = true;
        if (fail) {
            // proportional-fitting step  alpha += log(rhs / g)
            if (tid < m) sm.delta[tid] = log(rhs[tid] / sm.g[tid]);
            __syncthreads();
        }
        double dl = tid < m ? sm.delta[tid] : 0.0;
        if (!(dl == dl)) dl = 0.0;
        if (!slack) dl -= block_reduce_sum(tid < m ? dl : 0.0, red) / (double)m;
        const double dm = block_reduce_max(tid < m ? fabs(dl) : 0.0, red);
        // a full Newton step below 1e-11 in alpha: the weights cannot be improved at this quadrature accuracy
        if (!fail && dm < 1.0e-11) { status = GR_OK; it++; break; }
        if (dm > kFStepClamp) dl *= kFStepClamp / dm;
        // second-order size of the step, sum_i g_i delta_i^2: what a full Newton step in alpha = log w leaves behind
        // (each flow g_i is a sum of terms exponential in alpha over positive normalisers, so the part of g the
        // linear model misses is of the order of g_i delta_i^2 per token)
        const double s2 = block_reduce_sum(tid < m ? sm.g[tid] * dl * dl : 0.0, red);
        if (tid < m) {
            sm.delta[tid] = dl;
            sm.alpha[tid] = fmin(fmax(sm.alpha[tid] + dl, -kFAlphaClamp), kFAlphaClamp);
        }
        __syncthreads();
        // Stop on a predicted residual, without another evaluation, after a step from a point evaluated on the full
        // grid.  Two forms.  (i) The step is small: the residual it leaves is bounded by a small multiple of s2
        // (measured on every benchmark shape and at target temperatures down to 0.3, 2300 full-grid steps: next residual
        // <= 8.5 s2 + the quadrature floor of ~3e-9, median 0.15 s2); with 10 s2 below the tolerance the step is taken,
        // and the reported norm is 3 s2.  (ii) The last full step on this grid contracted the residual by rho < 0.1:
        // the next one is taken to contract no worse (Newton's contraction improves as it converges, and where it
        // converges only linearly, by 0.03 - 0.06 per step on systems with a small pivot, this is what happens), so
        // 3 rho r_k below the tolerance stops; the reported norm is rho r_k.  This form serves tolerances near the
        // quadrature floor, where s2 is too coarse.
        // Neither is trusted when the factorisation cancelled all but a few percent of some diagonal entry: with
        // weights of 1e5 and more the fp32 system stops producing Newton steps, the residual stays where it is while
        // the steps, and with them s2, shrink; every such case measured had a relative pivot below 4e-3, every other
        // above 3e-2.
        const bool by_step = !coarse && dm <= kFPredictStep && kFPredictSafety * s2 < tol;
        const bool by_ratio = rho < 0.1 && dm <= kFStepClamp && kFRatioSafety * rho * rn < tol;
        if (!fail && (by_step || by_ratio)
            && fast_relative_pivot(sm, m, slack ? 0.0 : 1.0 / (double)m) > kFTrustPivot) {
            if (tid < m) sm.w[tid] = exp(sm.alpha[tid]);
            __syncthreads();
            rn = by_step ? kFPredictBound * s2 : rho * rn;
            status = GR_OK; it++;
            predicted = true;
            break;
        }
    }
    if (status != GR_OK) {
        // not converged here: leave the last accepted point (the fp64 kernel's starting point)
        __syncthreads();
        if (tid < m) sm.w[tid] = exp(status == GR_NOT_CONVERGED ? sm.alpha_prev[tid] : sm.alpha[tid]);
        __syncthreads();
    }
    *gnorm = rn;
    *iters = it | (predicted ? kItersPredicted : 0);
    return status;
}

template <int NT, int TPL>
__global__ void __launch_bounds__(kFT, kFCtas)
fast_solve_kernel(const char* __restrict__ ws, char* __restrict__ params, int pstride, int kcap, int V, int n, int topk,
                  double temp_t, double temp_d, double tol, int max_iters, double qstep, double tau,
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
    if (kcap == 0 || wv.h->bad != 0 || wv.h->count <= 0) {
        if (tid == 0) write_no_rule(pv.h, n, wv.h->bad != 0, alpha_out, status_out, b);
        if (fused) {
            __syncthreads();
            fused_draw(fa, pv.h, b, n, smem_raw, GR_CHECK_FLAG);
        }
        return;
    }
    const int KP = kcap;
    FastLayout L(KP, NT);
    double* base = reinterpret_cast<double*>(smem_raw);
    FSm sm;
    int* const ck = GR_CHECK_FLAG;
    (void)ck;
    sm.d = GR_MKPTR(double, base + L.d, KP, ck); sm.tg = GR_MKPTR(double, base + L.tg, KP, ck);
    sm.p = GR_MKPTR(double, base + L.p, KP, ck); sm.r = GR_MKPTR(double, base + L.r, KP, ck);
    sm.key = GR_MKPTR(double, base + L.key, KP, ck);
    sm.psi = GR_MKPTR(double, base + L.psi, KP + 4, ck); sm.Dr = GR_MKPTR(double, base + L.Dr, KP + 4, ck);
    sm.alpha = GR_MKPTR(double, base + L.alpha, KP, ck); sm.alpha_prev = GR_MKPTR(double, base + L.alpha_prev, KP, ck);
    sm.delta = GR_MKPTR(double, base + L.delta, KP, ck); sm.w = GR_MKPTR(double, base + L.w, KP, ck);
    sm.g = GR_MKPTR(double, base + L.g, KP, ck); sm.g2 = GR_MKPTR(double, base + L.g2, KP, ck);
    sm.col = GR_MKPTR(double, base + L.col, kMP, ck);
    sm.gw = GR_MKPTR(double, base + L.gw, kFW * KP, ck); sm.g2w = GR_MKPTR(double, base + L.g2w, kFW * KP, ck);
    sm.tq = GR_MKPTR(double, base + L.tq, kFMaxNodes, ck); sm.cq = GR_MKPTR(double, base + L.cq, kFMaxNodes, ck);
    sm.scal = GR_MKPTR(double, base + L.scal, 48, ck);
    sm.J = GR_MKPTR(double, base + L.uni, L.uni_doubles, ck);
    sm.AS = GR_MKPTR(float, reinterpret_cast<float*>(base + L.uni), kJC * NT * kMS, ck);
    sm.HS = GR_MKPTR(float, reinterpret_cast<float*>(base + L.uni) + kJC * NT * kMS, kJC * NT * kMS, ck);
    sm.Jacc = GR_MKPTR(float, reinterpret_cast<float*>(smem_raw + L.jacc_bytes_off), kMP * kJS, ck);
    int* ib = reinterpret_cast<int*>(smem_raw + L.ints);
    sm.id = GR_MKPTR(int, ib, KP, ck); sm.blk = GR_MKPTR(int, ib + KP, KP, ck);
    sm.itmp = GR_MKPTR(int, ib + 2 * KP, KP, ck); sm.trunc = GR_MKPTR(int, ib + 3 * KP, KP, ck);
    sm.KP = KP;
    PrepSm ps;
    ps.d = sm.d; ps.tg = sm.tg; ps.p = sm.p; ps.r = sm.r; ps.key = sm.key; ps.psi = sm.psi; ps.Dr = sm.Dr;
    ps.id = sm.id; ps.blk = sm.blk; ps.itmp = sm.itmp; ps.red = sm.scal + SC_RED; ps.out3 = sm.scal + 16;
    const PrepResult pr = prep_instance(ps, wv, pv.h, V, n, topk, temp_t, temp_d);
    const int k = pr.k, jstar = pr.jstar;

    int status = GR_OK, iters_total = 0;
    double gnorm_total = 0.0;
    // Truncated variant (Algorithm 1 with an error threshold): every system is solved on its truncation set alone,
    // to gradient norm 5 tau; the other tokens keep weight 0.  The gathered arrays reuse what the preparation no
    // longer needs.
    const bool trunc = tau > 0.0;
    if (trunc) {
        truncation_sets(ps, sm.trunc, sm.itmp, k, jstar, n, tau);
        tol = 5.0 * tau;
    }
    GR_PTR(double) dT = sm.key; GR_PTR(double) rT = sm.psi; GR_PTR(int) tmap = sm.itmp;
    if (tid < k) pv.w[tid] = trunc ? 0.0 : 1.0;
    // with the drafted tuple at hand only the system it selects is solved
    const int sel = fused ? selected_system(fa.draft + (size_t)b * n, n, k, jstar, sm.id, sm.blk, &s_sel) : -2;
    bool skipped = false;
    if (jstar > 0 && sel >= 0) skipped = true;
    if (jstar > 0 && sel < 0) {
        double gn = 0.0; int it = 0;
        if (!trunc) {
            const int st = fast_system<NT, TPL>(sm, jstar, n, sm.d, sm.tg, 0.0, 1, tol, max_iters, qstep, &gn, &it);
            if (st != GR_OK) status = kNeedFallback;
            if (tid < jstar) pv.w[tid] = sm.w[tid];
        } else {
            const int mT = gather_truncated(sm.trunc, 0, jstar, sm.d, sm.tg, dT, rT, tmap, &s_sel);
            if (mT > 0) {
                const int st = fast_system<NT, TPL>(sm, mT, n, dT, rT, 0.0, 1, tol, max_iters, qstep, &gn, &it);
                if (st != GR_OK) status = kNeedFallback;
                if (tid < mT) pv.w[tmap[tid]] = sm.w[tid];
            }
        }
        gnorm_total += gn; iters_total = add_iters(iters_total, it);
        __syncthreads();
    }
    int lo = jstar;
    while (lo < k && status == GR_OK) {
        int hi = lo;
        const int bk = sm.blk[lo];
        while (hi + 1 < k && sm.blk[hi + 1] == bk) hi++;
        const int m = hi - lo + 1;
        const bool wanted = sel == -2 || sel == bk;
        if (!trunc) {
            if (m >= 2 && !wanted) skipped = true;
            if (m >= 2 && wanted) {
                double gn; int it;
                const int st = fast_system<NT, TPL>(sm, m, n, sm.d + lo, sm.p + lo, sm.Dr[lo], 0, tol, max_iters, qstep,
                                                    &gn, &it);
                if (st != GR_OK) status = kNeedFallback;
                gnorm_total += gn; iters_total = add_iters(iters_total, it);
                if (tid < m) pv.w[lo + tid] = sm.w[tid];
                __syncthreads();
            }
        } else {
            // tuples counted: those inside (H* u T)^n, so the mass above the block is drf(H*) plus the T-part of the
            // higher-ratio outer blocks
            double hT = sm.Dr[jstar];
            for (int j = jstar; j < lo; j++) hT += sm.trunc[j] ? sm.d[j] : 0.0;
            const int mT = gather_truncated(sm.trunc, lo, hi + 1, sm.d, sm.p, dT, rT, tmap, &s_sel);
            if (mT == 1 && tid == 0) pv.w[tmap[0]] = 1.0;
            if (mT >= 2 && !wanted) skipped = true;
            if (mT >= 2 && wanted) {
                double gn; int it;
                const int st = fast_system<NT, TPL>(sm, mT, n, dT, rT, hT, 0, tol, max_iters, qstep, &gn, &it);
                if (st != GR_OK) status = kNeedFallback;
                gnorm_total += gn; iters_total = add_iters(iters_total, it);
                if (tid < mT) pv.w[tmap[tid]] = sm.w[tid];
            }
            __syncthreads();
        }
        lo = hi + 1;
    }
    if (status == GR_OK && skipped) status = GR_PARTIAL_RULE;
    write_rule(ps, pv, KP, pr, n, status, gnorm_total, iters_total, alpha_out, status_out, b, GR_CHECK_FLAG,
               wv.h->check);
    if (fused && status != kNeedFallback) {
        __syncthreads();                       // the rule this CTA wrote is visible to its first warp
        fused_draw(fa, pv.h, b, n, smem_raw + L.uni * 8, GR_CHECK_FLAG);
    }
}

template <int NT, int TPL>
int launch_fast_t(const char* ws, char* params, int pstride, int kcap, int V, int n, int topk, double temp_t,
                         double temp_d, double tol, int max_iters, double qstep, double tau, int batch, float* alpha_out,
                         int* status_out, FusedArgs fa, cudaStream_t st)
{
    const int smem = fast_smem_bytes(kcap, NT);
    // function attributes belong to the device: set once per device
    static bool configured[kMaxDevices] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return GR_E_LAUNCH; }
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(fast_solve_kernel<NT, TPL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kMP == 64 ? 96 * 1024 : 200 * 1024) != cudaSuccess)
            return GR_E_LAUNCH;
        // the CTAs are small: ask for the largest shared-memory carve-out so that kFCtas of them fit on an SM
        if (cudaFuncSetAttribute(fast_solve_kernel<NT, TPL>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 cudaSharedmemCarveoutMaxShared) != cudaSuccess)
            return GR_E_LAUNCH;
        configured[dev] = true;
    }
    fast_solve_kernel<NT, TPL><<<batch, kFT, smem, st>>>(ws, params, pstride, kcap, V, n, topk, temp_t, temp_d, tol,
                                                         max_iters, qstep, tau, alpha_out, status_out, fa);
    return GR_OK;
}

// One translation unit per series length instantiates its kernels (they compile in parallel).
#define GR_FAST_ARGS                                                                                              \
    const char *ws, char *params, int pstride, int kcap, int V, int n, int topk, double temp_t, double temp_d,   \
        double tol, int max_iters, double qstep, double tau, int batch, float *alpha_out, int *status_out,       \
        FusedArgs fa, cudaStream_t st
#define GR_FAST_PASS ws, params, pstride, kcap, V, n, topk, temp_t, temp_d, tol, max_iters, qstep, tau, batch, alpha_out, status_out, fa, st
#define GR_FAST_INSTANTIATE(NT)                                                                \
    int launch_fast_n##NT(GR_FAST_ARGS) {                                                       \
        return kcap <= 32 * (kRL - 1) ? launch_fast_t<NT, kRL - 1>(GR_FAST_PASS)                    \
                                      : launch_fast_t<NT, kRL>(GR_FAST_PASS);                       \
    }

}  // namespace GR_FAST_NS
}  // namespace gr
