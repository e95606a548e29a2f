// Steps shared by the two solve kernels (one CTA per instance, any block size that is a multiple of 32
// and at least the support size + 1): distributions on the support, ratio order, subset selection,
// outer residuals and blocks; writing the rule into the params block.
#pragma once
#include "gr_common.cuh"

namespace gr {

constexpr int kNeedFallback = 100;   // internal status: the fast kernel asks the robust kernel to redo the instance

// CTA-wide reductions; `scratch` needs one double per warp.  Every thread gets the result.
__device__ inline double block_reduce_max(double v, GR_PTR(double) scratch) {
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
    const int nw = blockDim.x >> 5;
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    double r = scratch[0];
    for (int i = 1; i < nw; i++) r = fmax(r, scratch[i]);
    return r;
}
__device__ inline double block_reduce_sum(double v, GR_PTR(double) scratch) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const int nw = blockDim.x >> 5;
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    double r = 0.0;
    for (int i = 0; i < nw; i++) r += scratch[i];
    return r;
}

// shared-memory arrays of the preparation (KP entries each; psi and Dr: KP + 4)
struct PrepSm {
    GR_PTR(double) d, tg, p, r, key, psi, Dr;
    GR_PTR(int) id, blk, itmp;
    GR_PTR(double) red;     // one double per warp of reduction scratch
    GR_PTR(double) out3;    // 3 doubles: jstar, nblocks, alpha*
};
struct PrepResult { int k, jstar, nblocks; double alpha_star, lse_t; };

struct WsView { const WsHeader* h; GR_PTR(const int) id; GR_PTR(const float) dl; GR_PTR(const float) tl; };
__device__ inline WsView view_ws(const char* ws, long long b, int* flag = nullptr) {
    WsView v;
    v.h = reinterpret_cast<const WsHeader*>(ws + (size_t)b * ws_stride());
    const int* ids = reinterpret_cast<const int*>((const char*)v.h + sizeof(WsHeader));
    const float* dls = reinterpret_cast<const float*>(ids + kMaxSupport);
    v.id = GR_MKPTR(const int, ids, kMaxSupport, flag);
    v.dl = GR_MKPTR(const float, dls, kMaxSupport, flag);
    v.tl = GR_MKPTR(const float, dls + kMaxSupport, kMaxSupport, flag);
    (void)flag;
    return v;
}

// Header of an instance for which no rule exists (support beyond the capacity, or unusable logits).
__device__ inline void write_no_rule(Header* h, int n, bool bad, float* alpha_out, int* status_out, long long b) {
    h->n = n; h->k = 0; h->jstar = 0; h->nblocks = 0;
    h->status = bad ? GR_BAD_LOGITS : GR_SUPPORT_TOO_LARGE;
    h->alpha_star = __longlong_as_double(0x7ff8000000000000ll);
    h->resid_total = 1.0; h->gnorm = 0.0; h->iters = 0;
    __threadfence();
    h->magic = kMagic;
    alpha_out[b] = __int_as_float(0x7fc00000);
    status_out[b] = h->status;
}

// Everything before the convex minimisation.  Every thread of the CTA calls it.
__device__ inline PrepResult prep_instance(const PrepSm& sm, const WsView& wv, Header* hdr, int V, int n, int topk,
                                           double temp_t, double temp_d)
{
    const int tid = threadIdx.x;
    const int kfull = (topk <= 0 || topk >= V) ? V : topk;
    const int k = wv.h->count;
    double lse_t = wv.h->lse_t;
    // ---- distributions on the support (App. A; App. N): fp64 from the fp32 / bf16 logits
    double a_i = 0.0, b_i = 0.0;
    int my_id = 0;
    if (tid < k) {
        my_id = wv.id[tid];
        a_i = (double)wv.tl[tid] / temp_t;
        b_i = (double)wv.dl[tid] / temp_d;
    }
    const double bmax = block_reduce_max(tid < k ? b_i : -1.0e300, sm.red);
    const double bsum = block_reduce_sum(tid < k ? exp(b_i - bmax) : 0.0, sm.red);
    const double lse_d = bmax + log(bsum);
    if (kfull == V) {
        // the support is the whole vocabulary: normalise the target in fp64 over these same entries, so that
        // it sums to one to rounding (the streaming kernel's fp32 sum is only good to ~1e-7, which would
        // leave the outermost block's flows inconsistent with the mass of the tuples that feed them)
        const double amax = block_reduce_max(tid < k ? a_i : -1.0e300, sm.red);
        const double asum = block_reduce_sum(tid < k ? exp(a_i - amax) : 0.0, sm.red);
        lse_t = amax + log(asum);
        if (tid == 0) hdr->lse_t = lse_t;
    }
    // ---- ratio order: decreasing log-ratio key, equal keys by smaller id (Sec. 5.1)
    if (tid < k) { sm.key[tid] = b_i - a_i; sm.itmp[tid] = my_id; }
    __syncthreads();
    if (tid < k) {
        const double ky = sm.key[tid];
        int rank = 0;
        for (int j = 0; j < k; j++) {
            const double kj = sm.key[j];
            rank += (kj > ky || (kj == ky && sm.itmp[j] < my_id)) ? 1 : 0;
        }
        sm.id[rank] = my_id;
        sm.tg[rank] = exp(a_i - lse_t);
        sm.d[rank] = exp(b_i - lse_d);
    }
    __syncthreads();
    // ---- prefix sums in order, psi along the chain, H* and alpha* (Eq. "subset-select")
    if (tid == 0) {
        // (summed in order, one after the other, four loads ahead of the stores)
        double Tg = 0.0, Dr = 0.0;
        sm.psi[0] = 0.0; sm.Dr[0] = 0.0;
        for (int j0 = 0; j0 < k; j0 += 4) {
            double tv[4], dv[4];
#pragma unroll
            for (int u = 0; u < 4; u++) {
                const bool in = j0 + u < k;
                tv[u] = in ? sm.tg[j0 + u] : 0.0; dv[u] = in ? sm.d[j0 + u] : 0.0;
            }
#pragma unroll
            for (int u = 0; u < 4; u++) {
                const int j = j0 + u + 1;
                if (j <= k) {
                    Tg += tv[u]; Dr += dv[u];
                    if (j == k) { Dr = 1.0; if (kfull == V) Tg = 1.0; }   // both distributions are normalised
                    sm.psi[j] = Tg; sm.Dr[j] = Dr;
                }
            }
        }
    }
    __syncthreads();
    for (int j = 1 + tid; j <= k; j += blockDim.x) {
        const double base = sm.Dr[j];
        double pw = 1.0, sq = base;
        for (int e = n; e > 0; e >>= 1) { if (e & 1) pw *= sq; sq *= sq; }
        sm.psi[j] = sm.psi[j] - pw;
    }
    __syncthreads();
    // first strict minimum of psi (H* = the prefix up to it), every thread for itself
    int jstar = 0; double best = 0.0;
    for (int j = 1; j <= k; j++) {
        const double v = sm.psi[j];
        if (v < best) { best = v; jstar = j; }
    }
    // ---- outer residuals by cumulative minima along the increasing-ratio chain; blocks end at
    //      every new strict minimum (Sec. 6.1, Thm "polymatroid", Lemma "q-convex").  One position per thread:
    //      the running minimum that reaches a position is the minimum of psi over the positions above it
    //      (exact in any order), and its block number counts the strict minima above it.
    for (int pos = tid; pos < k; pos += blockDim.x) {
        if (pos < jstar) {
            sm.p[pos] = sm.tg[pos]; sm.r[pos] = 0.0; sm.blk[pos] = -1;
        } else {
            double m_prev = sm.psi[k];
            int blk = 0;
            for (int j = k - 1; j > pos; j--) {
                const double c = sm.psi[j];
                if (c < m_prev) { m_prev = c; blk++; }
            }
            const double c = sm.psi[pos];
            const double rr = c < m_prev ? m_prev - c : 0.0;
            sm.r[pos] = rr;
            sm.p[pos] = sm.tg[pos] - rr;
            sm.blk[pos] = blk;
            if (pos == jstar) {
                // the lowest position of the chain closes the last block: it is open unless this position is a record
                sm.out3[1] = (double)(blk + 1);
            }
        }
    }
    if (tid == 0) {
        sm.out3[0] = (double)jstar;
        if (jstar >= k) sm.out3[1] = 0.0;
        sm.out3[2] = 1.0 + best;
    }
    __syncthreads();
    PrepResult pr;
    pr.k = k; pr.jstar = (int)sm.out3[0]; pr.nblocks = (int)sm.out3[1]; pr.alpha_star = sm.out3[2]; pr.lse_t = lse_t;
    __syncthreads();
    return pr;
}

// Truncation sets of the truncated variant (Sec. 6.2 "tunable errors", Sec. 6.3, Algorithm 1): the fewest tokens with
//   inner:  T in H*,       gamma_T   = drf(H*)^n - drf(T)^n      <= tau,
//   outer:  T in V \ H*,   epsilon_T = 1 - (drf(H*) + drf(T))^n  <= tau,
// i.e. tokens in decreasing drf (equal drf: smaller id first) until the bound holds.  in_T[pos] = 1 / 0 for the
// k support positions (ratio order); scratch: k ints.  Every thread of the CTA calls it (blockDim.x >= k).
__device__ inline void truncation_sets(const PrepSm& sm, GR_PTR(int) in_T, GR_PTR(int) scratch, int k, int jstar, int n,
                                       double tau)
{
    const int tid = threadIdx.x;
    if (tid < k) {
        // rank inside the own group (H* or the outer support) by (drf descending, id ascending)
        const bool inner = tid < jstar;
        const int lo = inner ? 0 : jstar, hi = inner ? jstar : k;
        const double dv = sm.d[tid];
        const int iv = sm.id[tid];
        int rank = 0;
        for (int j = lo; j < hi; j++) {
            const double dj = sm.d[j];
            rank += (dj > dv || (dj == dv && sm.id[j] < iv)) ? 1 : 0;
        }
        scratch[lo + rank] = tid;          // position of the group's rank-th token
        in_T[tid] = 0;
    }
    __syncthreads();
    if (tid == 0) {
        double D = 0.0;
        for (int j = 0; j < jstar; j++) D += sm.d[j];
        auto powi = [](double x, int e) { double r = 1.0; while (e > 0) { if (e & 1) r *= x; x *= x; e >>= 1; } return r; };
        const double Dn = powi(D, n);
        double c = 0.0, gam = Dn;
        for (int q = 0; q < jstar && gam > tau; q++) {
            const int pos = scratch[q];
            c += sm.d[pos]; in_T[pos] = 1;
            gam = Dn - powi(c, n);
        }
        c = D;
        double eps = 1.0 - Dn;
        for (int q = jstar; q < k && eps > tau; q++) {
            const int pos = scratch[q];
            c += sm.d[pos]; in_T[pos] = 1;
            eps = 1.0 - powi(c, n);
        }
    }
    __syncthreads();
}

// The T-part of positions lo .. hi-1 gathered into contiguous arrays (draft masses, right-hand sides, positions);
// returns how many.  Every thread of the CTA calls it; `count` is one int of shared memory.
__device__ inline int gather_truncated(GR_PTR(const int) in_T, int lo, int hi, GR_PTR(const double) d,
                                       GR_PTR(const double) rhs, GR_PTR(double) dT, GR_PTR(double) rT, GR_PTR(int) map,
                                       int* count)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        int m = 0;
        for (int j = lo; j < hi; j++)
            if (in_T[j]) { dT[m] = d[j]; rT[m] = rhs[j]; map[m] = j; m++; }
        *count = m;
    }
    __syncthreads();
    return *count;
}

// Rule arrays (except w, which the solvers write as they go) and the header.
// `check_flag` / `check_before`: the bounds-checked build's per-CTA flag and what the streaming kernel reported for
// the row (nullptr / 0 otherwise): a skipped access turns the status into GR_CHECK_FAILED.
__device__ inline void write_rule(const PrepSm& sm, const ParamView& pv, int KP, const PrepResult& pr, int n,
                                  int status, double gnorm, int iters, float* alpha_out, int* status_out, long long b,
                                  const int* check_flag = nullptr, int check_before = 0)
{
    const int tid = threadIdx.x;
    for (int j = tid; j < KP; j += blockDim.x) {
        const bool in = j < pr.k;
        pv.id[j] = in ? sm.id[j] : -1;
        pv.blk[j] = in ? sm.blk[j] : -2;
        pv.r[j] = in ? sm.r[j] : 0.0;
        pv.p[j] = in ? sm.p[j] : 0.0;
        if (!in) pv.w[j] = 0.0;
    }
    __syncthreads();
    if (tid == 0) {
        if (check_before || (check_flag && *check_flag)) status = GR_CHECK_FAILED;
        Header* h = pv.h;
        h->n = n; h->k = pr.k; h->jstar = pr.jstar; h->nblocks = pr.nblocks; h->status = status;
        h->alpha_star = pr.alpha_star;
        h->resid_total = 1.0 - pr.alpha_star;
        h->gnorm = gnorm; h->iters = iters;
        __threadfence();
        h->magic = kMagic;
        alpha_out[b] = (float)pr.alpha_star;
        status_out[b] = status == kNeedFallback ? GR_NOT_CONVERGED : status;
    }
}

}  // namespace gr
