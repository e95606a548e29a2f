// Stand-alone verification kernel (one warp per instance) and the kernel that copies a rule out of the params block.
#include "gr_verify.cuh"

namespace gr {

constexpr int kVerifyWarps = 4;

__global__ void __launch_bounds__(kVerifyWarps * 32)
verify_kernel(const char* __restrict__ params, const int* __restrict__ draft, const float* __restrict__ uni, int batch,
              int* __restrict__ out_token, unsigned char* __restrict__ out_acc, int* __restrict__ status_out)
{
    __shared__ double s_scratch[kVerifyWarps][kVerifyScratchBytes / 8];
    GR_CHECK_FLAG_DECL;
    GR_CHECK_FLAG_INIT;
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
    }
    if (status == GR_OK)
        verify_instance(h, draft + (size_t)b * h->n, uni + 2 * (size_t)b, lane,
                        verify_scratch(s_scratch[wib], GR_CHECK_FLAG), false, token, accepted, status);
    __syncwarp();
    if (GR_CHECK_VALUE) status = GR_CHECK_FAILED;      // (the flag is shared by the CTA's four instances)
    if (lane == 0) {
        out_token[b] = token;
        out_acc[b] = (unsigned char)accepted;
        status_out[b] = status;
    }
}

// The slice pi(.|omega) of every instance as the verification code computes it (one warp per instance), for
// inspection: entry s of an instance's row belongs to drafted token s; repeats of an earlier token get id -1.
__global__ void __launch_bounds__(kVerifyWarps * 32)
read_slice_kernel(const char* __restrict__ params, const int* __restrict__ draft, int batch, int nmax,
                  int* __restrict__ U, double* __restrict__ pi, double* __restrict__ rho, int* __restrict__ status_out)
{
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int b = blockIdx.x * kVerifyWarps + wib;
    if (b >= batch) return;
    const Header* h0 = reinterpret_cast<const Header*>(params);
    int status = GR_OK;
    const Header* h = nullptr;
    if (h0->magic != kMagic || h0->stride <= 0) {
        status = GR_STALE_PARAMS;
    } else {
        h = reinterpret_cast<const Header*>(params + (size_t)b * h0->stride);
        if (h->magic != kMagic) status = GR_STALE_PARAMS;
    }
    SliceLane sl;
    sl.uniq = false; sl.inner = false; sl.pi = 0.0; sl.rho = 0.0;
    int tok = -1, n = 0;
    if (status == GR_OK) {
        n = h->n < nmax ? h->n : nmax;
        status = h->status;
        if (status == GR_OK || status == GR_NOT_CONVERGED) {
            ParamView pv = view_params((void*)h, h->kcap, h->V, nullptr);
            tok = lane < h->n ? draft[(size_t)b * h->n + lane] : -1;
            const int rs = h->k > 0 ? slice_instance(h, pv, tok, lane, sl) : GR_SUPPORT_TOO_LARGE;
            if (rs != GR_OK) { status = rs; sl.uniq = false; sl.pi = 0.0; sl.rho = 0.0; }
        }
    }
    if (lane < nmax) {
        const bool on = lane < n && sl.uniq;
        U[(size_t)b * nmax + lane] = on ? tok : -1;
        pi[(size_t)b * nmax + lane] = on ? sl.pi : 0.0;
    }
    if (lane == 0) { rho[b] = sl.rho; status_out[b] = status; }
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
void launch_read_slice(const char* params, const int* draft, int batch, int n, int* U, double* pi, double* rho,
                       int* status, cudaStream_t st)
{
    const int blocks = (batch + kVerifyWarps - 1) / kVerifyWarps;
    read_slice_kernel<<<blocks, kVerifyWarps * 32, 0, st>>>(params, draft, batch, n, U, pi, rho, status);
}
void launch_read_rule(const char* params, int batch, int kcap, int* ids, int* block, double* w, double* resid,
                      double* flow, double* header, cudaStream_t st)
{
    read_rule_kernel<<<batch, 128, 0, st>>>(params, batch, kcap, ids, block, w, resid, flow, header);
}

}  // namespace gr
