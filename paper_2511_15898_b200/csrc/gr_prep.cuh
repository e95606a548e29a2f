// Steps shared by the two solve kernels (one CTA per instance, any block size that is a multiple of 32
// and at least the support size + 1): distributions on the support, ratio order, subset selection,
// outer residuals and blocks; writing the rule into the params block.
#pragma once
#include "gr_common.cuh"

namespace gr {

constexpr int kNeedFallback = 100;   // internal status: the fast kernel asks the robust kernel to redo the instance

// CTA-wide reductions; `scratch` needs one double per warp.  Every thread gets the result.
__device__ inline double block_reduce_max(double v, double* scratch) {
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
    const int nw = blockDim.x >> 5;
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    double r = scratch[0];
    for (int i = 1; i < nw; i++) r = fmax(r, scratch[i]);
    return r;
}
__device__ inline double block_reduce_sum(double v, double* scratch) {
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
    double *d, *tg, *p, *r, *key, *psi, *Dr;
    int *id, *blk, *itmp;
    double* red;     // one double per warp of reduction scratch
    double* out3;    // 3 doubles: jstar, nblocks, alpha*
};
struct PrepResult { int k, jstar, nblocks; double alpha_star, lse_t; };

struct WsView { const WsHeader* h; const int* id; const float* dl; const float* tl; };
__device__ inline WsView view_ws(const char* ws, long long b) {
    WsView v;
    v.h = reinterpret_cast<const WsHeader*>(ws + (size_t)b * ws_stride());
    v.id = reinterpret_cast<const int*>((const char*)v.h + sizeof(WsHeader));
    v.dl = reinterpret_cast<const float*>(v.id + kMaxSupport);
    v.tl = v.dl + kMaxSupport;
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
        double Tg = 0.0, Dr = 0.0;
        sm.psi[0] = 0.0; sm.Dr[0] = 0.0;
        for (int j = 1; j <= k; j++) {
            Tg += sm.tg[j - 1]; Dr += sm.d[j - 1];
            if (j == k) { Dr = 1.0; if (kfull == V) Tg = 1.0; }   // both distributions are normalised
            sm.psi[j] = Tg; sm.Dr[j] = Dr;
        }
    }
    __syncthreads();
    for (int j = 1 + tid; j <= k; j += blockDim.x) sm.psi[j] = sm.psi[j] - pow(sm.Dr[j], (double)n);
    __syncthreads();
    if (tid == 0) {
        int jstar = 0; double best = 0.0;
        for (int j = 1; j <= k; j++) if (sm.psi[j] < best) { best = sm.psi[j]; jstar = j; }
        // ---- outer residuals by cumulative minima along the increasing-ratio chain; blocks end at
        //      every new strict minimum (Sec. 6.1, Thm "polymatroid", Lemma "q-convex")
        for (int j = 0; j < jstar; j++) { sm.p[j] = sm.tg[j]; sm.r[j] = 0.0; sm.blk[j] = -1; }
        double m_prev = sm.psi[k];
        int blk = 0, open = 0;
        for (int s = 1; s <= k - jstar; s++) {
            const int pos = k - s;
            const double c = sm.psi[k - s];
            const bool record = c < m_prev;
            const double mm = record ? c : m_prev;
            sm.r[pos] = m_prev - mm;
            sm.p[pos] = sm.tg[pos] - sm.r[pos];
            sm.blk[pos] = blk; open = 1;
            if (record) { blk++; open = 0; }
            m_prev = mm;
        }
        sm.out3[0] = (double)jstar;
        sm.out3[1] = (double)(blk + open);
        sm.out3[2] = 1.0 + best;
    }
    __syncthreads();
    PrepResult pr;
    pr.k = k; pr.jstar = (int)sm.out3[0]; pr.nblocks = (int)sm.out3[1]; pr.alpha_star = sm.out3[2]; pr.lse_t = lse_t;
    __syncthreads();
    return pr;
}

// Rule arrays (except w, which the solvers write as they go) and the header.
__device__ inline void write_rule(const PrepSm& sm, const ParamView& pv, int KP, const PrepResult& pr, int n,
                                  int status, double gnorm, int iters, float* alpha_out, int* status_out, long long b)
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
