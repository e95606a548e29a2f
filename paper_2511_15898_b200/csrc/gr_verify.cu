// Slice of the transport for the drafted tuple and the accept / resample draw
// (Eq. "cases", Eq. "approx-c", "normalized" in Algorithm 1; App. A steps 3-4).
// One warp per instance.
#include "gr_common.cuh"

namespace gr {

constexpr int kVerifyWarps = 4;

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
__device__ int resample_draw(const Header* h, const ParamView& pv, int k, double frac, int lane,
                             int* l_id, double* l_r, int* s_id, double* s_p)
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
    // exact pass: every lane owns a contiguous piece of the chunk
    const int len = ce - cb;
    const int per = (len + 31) / 32;
    const int b0 = cb + lane * per, b1 = min(ce, b0 + per);
    double mysum = 0.0;
    for (int i = b0; i < b1; i++) {
        double res = exp((double)load_logit_dyn(row, dtype, i) / T - lse);
        for (int s = 0; s < nl; s++) if (l_id[s] == i) res = l_r[s];
        mysum += res;
    }
    const double inc = warp_incl_scan(mysum, lane);
    const double want = before < 0.0 ? 1.0e300 : thr - before;
    const unsigned hit = __ballot_sync(0xffffffffu, inc > want);
    const unsigned posl = __ballot_sync(0xffffffffu, mysum > 0.0);
    int owner = hit ? __ffs(hit) - 1 : (posl ? 31 - __clz(posl) : -1);
    if (owner < 0) return -1;
    int token = -1;
    if (lane == owner) {
        double acc = inc - mysum;
        int lastp = -1;
        for (int i = b0; i < b1; i++) {
            double res = exp((double)load_logit_dyn(row, dtype, i) / T - lse);
            for (int s = 0; s < nl; s++) if (l_id[s] == i) res = l_r[s];
            acc += res;
            if (res > 0.0) lastp = i;
            if (acc > want) { token = i; break; }
        }
        if (token < 0) token = lastp;
    }
    return __shfl_sync(0xffffffffu, token, owner);
}

__global__ void __launch_bounds__(kVerifyWarps * 32)
verify_kernel(const char* __restrict__ params, const int* __restrict__ draft, const float* __restrict__ uni, int batch,
              int* __restrict__ out_token, unsigned char* __restrict__ out_acc, int* __restrict__ status_out)
{
    __shared__ int s_lid[kVerifyWarps][kMaxSupport];
    __shared__ double s_lr[kVerifyWarps][kMaxSupport];
    __shared__ int s_sid[kVerifyWarps][kMaxSupport];
    __shared__ double s_sp[kVerifyWarps][kMaxSupport];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int b = blockIdx.x * kVerifyWarps + wib;
    if (b >= batch) return;
    const Header* h0 = reinterpret_cast<const Header*>(params);
    int token = -1, accepted = 0, status = GR_OK;
    const Header* h = nullptr;
    if (h0->magic != kMagic || h0->stride <= 0) {
        status = GR_STALE_PARAMS;
    } else {
        h = reinterpret_cast<const Header*>(params + (size_t)b * h0->stride);
        if (h->magic != kMagic) status = GR_STALE_PARAMS;
        else if (h->status == GR_BAD_LOGITS) status = GR_BAD_LOGITS;
    }
    if (status == GR_OK) {
        ParamView pv = view_params((void*)h, h->kcap);
        const int n = h->n, k = h->k, jstar = h->jstar;
        const double u0 = (double)uni[2 * (size_t)b], u1 = (double)uni[2 * (size_t)b + 1];
        const int tok = lane < n ? draft[(size_t)b * n + lane] : -1;
        if (k == 0) {
            // no rule was solved: emit a sample of the target distribution itself
            status = h->status;
            token = resample_draw(h, pv, 0, u1, lane, s_lid[wib], s_lr[wib], s_sid[wib], s_sp[wib]);
            accepted = __any_sync(0xffffffffu, lane < n && tok == token) ? 1 : 0;
            if (token < 0) accepted = 0;
        } else {
            status = h->status;
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
            if (missing) {
                status = GR_DRAFT_OUT_OF_SUPPORT;
            } else {
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
                const double pi = wv / W;
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
                    token = resample_draw(h, pv, k, u1, lane, s_lid[wib], s_lr[wib], s_sid[wib], s_sp[wib]);
                    accepted = 0;
                }
            }
        }
    }
    if (lane == 0) {
        out_token[b] = token;
        out_acc[b] = (unsigned char)accepted;
        status_out[b] = status;
    }
}

// copies the rule out of the params block into plain arrays
__global__ void read_rule_kernel(const char* __restrict__ params, int batch, int kcap_out, int* ids, int* block,
                                 double* w, double* resid, double* flow, double* header)
{
    const int b = blockIdx.x;
    const Header* h0 = reinterpret_cast<const Header*>(params);
    if (h0->magic != kMagic || h0->stride <= 0) {
        if (header && threadIdx.x < 8) header[(size_t)b * 8 + threadIdx.x] = threadIdx.x == 7 ? (double)GR_STALE_PARAMS : 0.0;
        return;
    }
    const Header* h = reinterpret_cast<const Header*>(params + (size_t)b * h0->stride);
    ParamView pv = view_params((void*)h, h->kcap);
    const int k = h->k;
    for (int j = threadIdx.x; j < kcap_out; j += blockDim.x) {
        const bool in = j < k && j < h->kcap;
        const size_t o = (size_t)b * kcap_out + j;
        if (ids) ids[o] = in ? pv.id[j] : -1;
        if (block) block[o] = in ? pv.blk[j] : -2;
        if (w) w[o] = in ? pv.w[j] : 0.0;
        if (resid) resid[o] = in ? pv.r[j] : 0.0;
        if (flow) flow[o] = in ? pv.p[j] : 0.0;
    }
    if (header && threadIdx.x == 0) {
        double* o = header + (size_t)b * 8;
        o[0] = (double)k; o[1] = (double)h->jstar; o[2] = (double)h->nblocks; o[3] = h->alpha_star;
        o[4] = h->gnorm; o[5] = (double)h->iters; o[6] = h->lse_t; o[7] = (double)h->status;
    }
}

void launch_verify(const char* params, const int* draft, const float* uni, int batch, int* out_token,
                   unsigned char* out_acc, int* status, cudaStream_t st)
{
    const int blocks = (batch + kVerifyWarps - 1) / kVerifyWarps;
    verify_kernel<<<blocks, kVerifyWarps * 32, 0, st>>>(params, draft, uni, batch, out_token, out_acc, status);
}
void launch_read_rule(const char* params, int batch, int kcap, int* ids, int* block, double* w, double* resid,
                      double* flow, double* header, cudaStream_t st)
{
    read_rule_kernel<<<batch, 128, 0, st>>>(params, batch, kcap, ids, block, w, resid, flow, header);
}

}  // namespace gr
