// Slice of the transport for the drafted tuple and the accept / resample draw
// (Eq. "cases", Eq. "approx-c", "normalized" in Algorithm 1; App. A steps 3-4), as warp-level
// device code: one warp serves one instance.  Used by the stand-alone verify kernel and by the
// solve kernels when they are given the drafted tokens (fused solve + verify).
#pragma once
#include "gr_common.cuh"

namespace gr {

// What a solve kernel needs to finish an instance with its draw; draft == nullptr: not fused.
struct FusedArgs {
    const int* draft;          // [batch, n]
    const float* uni;          // [batch, 2]
    int* out_token;            // [batch]
    unsigned char* out_acc;    // [batch]
    int* vstatus;              // [batch]
};

// Shared-memory scratch of one verifying warp.
struct VerifyScratch {
    GR_PTR(int) l_id; GR_PTR(double) l_r; GR_PTR(int) s_id; GR_PTR(double) s_p;       // kMaxSupport entries each
    int* flag;                                              // bounds-checked build: where skipped accesses are reported
};
constexpr int kVerifyScratchBytes = kMaxSupport * 24;
// base: 8-byte aligned, kVerifyScratchBytes long
__device__ inline VerifyScratch verify_scratch(void* base, int* flag = nullptr) {
    VerifyScratch v;
    double* lr = reinterpret_cast<double*>(base);
    int* li = reinterpret_cast<int*>(lr + 2 * kMaxSupport);
    v.l_r = GR_MKPTR(double, lr, kMaxSupport, flag);
    v.s_p = GR_MKPTR(double, lr + kMaxSupport, kMaxSupport, flag);
    v.l_id = GR_MKPTR(int, li, kMaxSupport, flag);
    v.s_id = GR_MKPTR(int, li + kMaxSupport, kMaxSupport, flag);
    v.flag = flag;
    return v;
}

__device__ __forceinline__ double warp_sum(double v) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_incl_scan(double v, int lane) {
    for (int o = 1; o < 32; o <<= 1) {
        double t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// Inverse CDF of the resample distribution in ascending id order at `frac` of its total.
// Residual of id i: the outer residual r_i on support ids (0 on H*), tgt_i elsewhere.
// Two levels: per-chunk masses from the scan kernel's table minus the flow p_i of the
// support ids in the chunk, then an exact fp64 pass over the one chunk selected.
__device__ inline int resample_draw(const Header* h, const ParamView& pv, int k, double frac, int lane,
                             GR_PTR(int) l_id, GR_PTR(double) l_r, GR_PTR(int) s_id, GR_PTR(double) s_p)
{
    const int nch = h->nch, head = h->head, V = h->V, dtype = h->dtype;
    const double T = (double)h->temp_target, lse = h->lse_t;
    const void* row = h->q_row;
    // The total residual mass is known in closed form (1 - alpha*, or 1 when the target itself is sampled), so
    // one pass over the chunk masses finds the chunk.  The support's (id, flow) pairs are staged in shared memory.
    for (int j = lane; j < k; j += 32) { s_id[j] = pv.id[j]; s_p[j] = pv.p[j]; }
    __syncwarp();
    const double thr = frac * (k > 0 ? h->resid_total : 1.0);
    int sel = -1; double before = 0.0, run = 0.0;
    int last_pos_chunk = -1;
    for (int c0 = 0; c0 < nch && sel < 0; c0 += 32) {
        const int c = c0 + lane;
        double R = 0.0;
        if (c < nch) {
            const float2 ms = pv.chunk[c];
            R = (double)ms.y * exp((double)ms.x / T - lse);
            const int cb = chunk_begin(c, head), ce = chunk_end(c, head, nch, V);
            for (int j = 0; j < k; j++) { const int id = s_id[j]; if (id >= cb && id < ce) R -= s_p[j]; }
            if (R < 0.0) R = 0.0;
        }
        const double inc = warp_incl_scan(R, lane) + run;
        const unsigned hit = __ballot_sync(0xffffffffu, c < nch && inc > thr);
        const unsigned pos = __ballot_sync(0xffffffffu, c < nch && R > 0.0);
        if (pos) last_pos_chunk = c0 + 31 - __clz(pos);
        if (hit) {
            const int l = __ffs(hit) - 1;
            sel = c0 + l;
            before = __shfl_sync(0xffffffffu, inc - R, l);
        }
        run = __shfl_sync(0xffffffffu, inc, 31);
    }
    if (sel < 0) { sel = last_pos_chunk; before = -1.0; }   // rounding left the threshold above the total
    if (sel < 0) return -1;
    // support ids inside the selected chunk
    const int cb = chunk_begin(sel, head), ce = chunk_end(sel, head, nch, V);
    int nl = 0;
    for (int j0 = 0; j0 < k; j0 += 32) {
        const int j = j0 + lane;
        const int id = j < k ? pv.id[j] : -1;
        const bool in = id >= cb && id < ce;
        const unsigned mk = __ballot_sync(0xffffffffu, in);
        if (in) { const int s = nl + __popc(mk & ((1u << lane) - 1u)); l_id[s] = id; l_r[s] = pv.r[j]; }
        nl += __popc(mk);
    }
    __syncwarp();
    // exact pass over the chunk in id order, 32 consecutive ids at a time (one per lane): the first id whose running
    // total exceeds the threshold; the last id of positive residual when rounding left the threshold above the total
    const double want = before < 0.0 ? 1.0e300 : thr - before;
    double run2 = 0.0;
    int token = -1, lastp = -1;
    constexpr int kRows = 8;                 // rows of 32 ids whose logits are fetched together
    for (int g0 = cb; g0 < ce && token < 0; g0 += 32 * kRows) {
        float lg[kRows];
#pragma unroll
        for (int q = 0; q < kRows; q++) {
            const int i = g0 + 32 * q + lane;
            lg[q] = i < ce ? load_logit_dyn(row, dtype, i) : 0.f;
        }
#pragma unroll
        for (int q = 0; q < kRows; q++) {
            const int r0 = g0 + 32 * q;
            if (r0 < ce && token < 0) {
                const int i = r0 + lane;
                const bool in = i < ce;
                double res = 0.0;
                if (in) {
                    res = exp((double)lg[q] / T - lse);
                    for (int s2 = 0; s2 < nl; s2++) if (l_id[s2] == i) res = l_r[s2];
                }
                const double inc = warp_incl_scan(res, lane) + run2;
                const unsigned hit = __ballot_sync(0xffffffffu, in && inc > want);
                const unsigned posl = __ballot_sync(0xffffffffu, in && res > 0.0);
                if (posl) lastp = r0 + 31 - __clz(posl);
                if (hit) token = r0 + __ffs(hit) - 1;
                run2 = __shfl_sync(0xffffffffu, inc, 31);
            }
        }
    }
    return token >= 0 ? token : lastp;
}


// One lane's share of the slice pi(.|omega) (Eq. "cases", Eq. "approx-c", "normalized" in Algorithm 1): lane s < n
// holds drafted token s.  uniq: first occurrence of its token; pi: its probability (0 for repeats and for tokens
// outside the serving system); inner: every drafted token lies in H*; rho: mass of the resample segment.
struct SliceLane { bool uniq, inner; double pi, rho; };

// Slice of a solved instance (k > 0) for the drafted tuple, one warp; `tok` is this lane's drafted token (lanes >= n: any).
// Returns GR_OK, or GR_DRAFT_OUT_OF_SUPPORT when a drafted token is not in the support.
__device__ inline int slice_instance(const Header* h, const ParamView& pv, int tok, int lane, SliceLane& sl)
{
    const int n = h->n, k = h->k, jstar = h->jstar;
    sl.uniq = false; sl.inner = false; sl.pi = 0.0; sl.rho = 0.0;
    // position of every drafted token in the ratio order
    int pos = -1;
    for (int s = 0; s < n; s++) {
        const int ts = __shfl_sync(0xffffffffu, tok, s);
        int found = -1;
        for (int j0 = 0; j0 < k; j0 += 32) {
            const int j = j0 + lane;
            const unsigned mk = __ballot_sync(0xffffffffu, j < k && pv.id[j] == ts);
            if (mk) found = j0 + __ffs(mk) - 1;
        }
        if (lane == s) pos = found;
    }
    const bool missing = __any_sync(0xffffffffu, lane < n && pos < 0);
    if (missing) return GR_DRAFT_OUT_OF_SUPPORT;
    // distinct tokens in order of first occurrence; the lowest-ratio position met
    bool uniq = lane < n;
    int maxpos = lane < n ? pos : -1;
    for (int s = 0; s < n; s++) {
        const int ps = __shfl_sync(0xffffffffu, pos, s);
        if (lane > s && lane < n && pos == ps) uniq = false;
    }
    for (int o = 16; o > 0; o >>= 1) maxpos = max(maxpos, __shfl_xor_sync(0xffffffffu, maxpos, o));
    const bool inner = maxpos < jstar;
    double wv = 0.0;
    if (uniq) {
        if (inner) wv = pv.w[pos];
        else wv = (pv.blk[pos] == pv.blk[maxpos]) ? pv.w[pos] : 0.0;
    }
    const double W = warp_sum(wv) + (inner ? 1.0 : 0.0);
    sl.uniq = uniq; sl.inner = inner;
    if (W > 0.0) {
        sl.pi = wv / W;
    } else {
        // (truncated variant) every served token carries weight 0: they share the tuple equally
        const bool served = uniq && pv.blk[pos] == pv.blk[maxpos];
        const int cnt = __popc(__ballot_sync(0xffffffffu, served));
        sl.pi = served ? 1.0 / (double)cnt : 0.0;
    }
    sl.rho = inner ? 1.0 / W : 0.0;
    return GR_OK;
}

// The whole verification of one instance by one warp.  `h` is the instance's header (already checked to carry
// the magic number); a rule marked partial is accepted only from the kernel that solved it for these drafts.
__device__ inline void verify_instance(const Header* h, const int* draft_row, const float* uni_row, int lane,
                                       const VerifyScratch& vs, bool allow_partial, int& token, int& accepted,
                                       int& status)
{
    token = -1; accepted = 0;
    status = h->status;
    if (status == GR_BAD_LOGITS) return;
    if (status == GR_PARTIAL_RULE) {
        if (!allow_partial) return;
        status = GR_OK;
    }
    ParamView pv = view_params((void*)h, h->kcap, h->V, vs.flag);
    const int n = h->n, k = h->k;
    const double u0 = (double)uni_row[0], u1 = (double)uni_row[1];
    const int tok = lane < n ? draft_row[lane] : -1;
    if (k == 0) {
        // no rule was solved: emit a sample of the target distribution itself
        token = resample_draw(h, pv, 0, u1, lane, vs.l_id, vs.l_r, vs.s_id, vs.s_p);
        accepted = __any_sync(0xffffffffu, lane < n && tok == token) ? 1 : 0;
        if (token < 0) accepted = 0;
        return;
    }
    SliceLane sl;
    if (slice_instance(h, pv, tok, lane, sl) != GR_OK) { status = GR_DRAFT_OUT_OF_SUPPORT; return; }
    const bool uniq = sl.uniq, inner = sl.inner;
    const double pi = sl.pi;
    const double cum = warp_incl_scan(pi, lane);
    const unsigned hit = __ballot_sync(0xffffffffu, uniq && cum > u0);
    if (hit) {
        token = __shfl_sync(0xffffffffu, tok, __ffs(hit) - 1);
        accepted = 1;
    } else if (!inner) {
        const unsigned posm = __ballot_sync(0xffffffffu, uniq && pi > 0.0);
        token = __shfl_sync(0xffffffffu, tok, 31 - __clz(posm));
        accepted = 1;
    } else {
        token = resample_draw(h, pv, k, u1, lane, vs.l_id, vs.l_r, vs.s_id, vs.s_p);
        accepted = 0;
    }
}

// Which system the drafted tuple selects (Eq. "cases"): -1 the inner system (every drafted token in H*), b >= 0 the
// outer block b (the lowest-ratio block met), -2 when a drafted token is outside the support (then every system is
// solved and the draw reports the error).  Every thread of the CTA calls it; id / blk are in ratio order.
__device__ inline int selected_system(const int* draft_row, int n, int k, int jstar, GR_PTR(const int) sid,
                                      GR_PTR(const int) sblk, int* s_sel)
{
    const int tid = threadIdx.x;
    if (tid == 0) *s_sel = -1;
    __syncthreads();
    int missing = 0;
    if (tid < n) {
        const int t = draft_row[tid];
        int pos = -1;
        for (int j = 0; j < k; j++) if (sid[j] == t) pos = j;
        if (pos < 0) missing = 1; else atomicMax(s_sel, pos);
    }
    missing = __syncthreads_or(missing);
    const int maxpos = *s_sel;
    __syncthreads();
    if (missing || maxpos < 0) return -2;
    return maxpos < jstar ? -1 : sblk[maxpos];
}

// Draw of instance b by warp 0 of a solve kernel's CTA, after the rule (or the no-rule header) was written and the
// CTA synchronised.
__device__ inline void fused_draw(const FusedArgs& fa, const Header* h, long long b, int n, void* scratch,
                                  int* check_flag = nullptr)
{
    if (threadIdx.x >= 32) return;
    const int lane = threadIdx.x;
    int token, accepted, status;
    verify_instance(h, fa.draft + (size_t)b * n, fa.uni + 2 * (size_t)b, lane, verify_scratch(scratch, check_flag), true,
                    token, accepted, status);
    if (check_flag && *check_flag) status = GR_CHECK_FAILED;
    if (lane == 0) {
        fa.out_token[b] = token;
        fa.out_acc[b] = (unsigned char)accepted;
        fa.vstatus[b] = status;
    }
}

}  // namespace gr
