// Optimal acceptance alpha* = 1 + min_H psi(H) alone, for several draft counts n at once
// (Eq. "subset-select"; the prefix sums along the ratio order do not depend on n, only
// psi_j = Tg_j - Dr_j^n does).  One CTA per instance, after the streaming kernel.
#include "gr_prep.cuh"

namespace gr {

constexpr int kAlphaThreads = 128;
struct NList { int n[GR_MAX_ALPHA_N]; int count; };

__global__ void __launch_bounds__(kAlphaThreads)
alpha_kernel(const char* __restrict__ ws, int V, int topk, double temp_t, double temp_d, NList nl,
             float* __restrict__ alpha_out, int* __restrict__ status_out)
{
    __shared__ double s_key[kMaxSupport], s_tg[kMaxSupport], s_d[kMaxSupport], s_Tg[kMaxSupport + 1], s_Dr[kMaxSupport + 1];
    __shared__ int s_id[kMaxSupport];
    __shared__ double s_red[32];
    const int tid = threadIdx.x;
    const long long b = blockIdx.x;
    const WsView wv = view_ws(ws, b);
    const int k = wv.h->count;
    if (wv.h->bad != 0 || k <= 0) {
        if (tid < nl.count) alpha_out[(size_t)b * nl.count + tid] = __int_as_float(0x7fc00000);
        if (tid == 0) status_out[b] = wv.h->bad != 0 ? GR_BAD_LOGITS : GR_SUPPORT_TOO_LARGE;
        return;
    }
    const int kfull = (topk <= 0 || topk >= V) ? V : topk;
    double lse_t = wv.h->lse_t;
    // distributions on the support in fp64 (App. A; App. N), as in the solve kernels
    double a_i = 0.0, b_i = 0.0;
    int my_id = 0;
    if (tid < k) {
        my_id = wv.id[tid];
        a_i = (double)wv.tl[tid] / temp_t;
        b_i = (double)wv.dl[tid] / temp_d;
    }
    const double bmax = block_reduce_max(tid < k ? b_i : -1.0e300, GR_MKPTR(double, s_red, 32, nullptr));
    const double bsum = block_reduce_sum(tid < k ? exp(b_i - bmax) : 0.0, GR_MKPTR(double, s_red, 32, nullptr));
    const double lse_d = bmax + log(bsum);
    if (kfull == V) {
        const double amax = block_reduce_max(tid < k ? a_i : -1.0e300, GR_MKPTR(double, s_red, 32, nullptr));
        const double asum = block_reduce_sum(tid < k ? exp(a_i - amax) : 0.0, GR_MKPTR(double, s_red, 32, nullptr));
        lse_t = amax + log(asum);
    }
    // ratio order: decreasing log-ratio, equal keys by smaller id (Sec. 5.1)
    if (tid < k) { s_key[tid] = b_i - a_i; s_id[tid] = my_id; }
    __syncthreads();
    if (tid < k) {
        const double ky = s_key[tid];
        int rank = 0;
        for (int j = 0; j < k; j++) {
            const double kj = s_key[j];
            rank += (kj > ky || (kj == ky && s_id[j] < my_id)) ? 1 : 0;
        }
        s_tg[rank] = exp(a_i - lse_t);
        s_d[rank] = exp(b_i - lse_d);
    }
    __syncthreads();
    if (tid == 0) {
        double Tg = 0.0, Dr = 0.0;
        s_Tg[0] = 0.0; s_Dr[0] = 0.0;
        for (int j = 1; j <= k; j++) {
            Tg += s_tg[j - 1]; Dr += s_d[j - 1];
            if (j == k) { Dr = 1.0; if (kfull == V) Tg = 1.0; }   // both distributions are normalised
            s_Tg[j] = Tg; s_Dr[j] = Dr;
        }
    }
    __syncthreads();
    // one warp per draft count: min over the prefixes of Tg_j - Dr_j^n
    const int warp = tid >> 5, lane = tid & 31;
    for (int e = warp; e < nl.count; e += kAlphaThreads / 32) {
        const int n = nl.n[e];
        double best = 0.0;                       // psi of the empty prefix
        for (int j = 1 + lane; j <= k; j += 32) {
            double pw = 1.0, sq = s_Dr[j];
            for (int m = n; m > 0; m >>= 1) { if (m & 1) pw *= sq; sq *= sq; }
            best = fmin(best, s_Tg[j] - pw);
        }
        for (int o = 16; o > 0; o >>= 1) best = fmin(best, __shfl_xor_sync(0xffffffffu, best, o));
        if (lane == 0) alpha_out[(size_t)b * nl.count + e] = (float)(1.0 + best);
    }
    if (tid == 0) status_out[b] = GR_OK;
}

void launch_alpha(const char* ws, int V, int topk, double temp_t, double temp_d, const int* n_list, int n_count,
                  int batch, float* alpha_out, int* status_out, cudaStream_t st)
{
    NList nl;
    nl.count = n_count;
    for (int i = 0; i < GR_MAX_ALPHA_N; i++) nl.n[i] = i < n_count ? n_list[i] : 1;
    alpha_kernel<<<batch, kAlphaThreads, 0, st>>>(ws, V, topk, temp_t, temp_d, nl, alpha_out, status_out);
}

}  // namespace gr
