// Host side of the C interface declared in gr.h: argument checks and kernel launches.
#include <math.h>
#include "gr_host.h"

namespace gr {
// The fast kernel covers supports up to 128 tokens with n <= 16; everything else, and any instance the fast
// kernel could not finish, takes the robust kernel.
int launch_solve_any(const char* ws, char* params, int pstride, int kcap, int V, int n, int topk, double temp_t,
                     double temp_d, double tol, int max_iters, double qstep, double tau, int batch, int force_robust,
                     float* alpha_out, int* status_out, FusedArgs fa, cudaStream_t st)
{
    int rc = force_robust ? 1
                          : launch_fast(ws, params, pstride, kcap, V, n, topk, temp_t, temp_d, tol, max_iters, qstep,
                                        tau, batch, alpha_out, status_out, fa, st);
    if (rc < 0) return rc;
    // rc == 1: no fast variant, the robust kernel does everything; rc == 0: it redoes what the fast one flagged
    return launch_solve(ws, params, pstride, kcap, V, n, topk, temp_t, temp_d, tol, max_iters, qstep, tau, batch,
                        rc == 0 ? 1 : 0, alpha_out, status_out, fa, st);
}

static bool shape_ok(int V, int n, int batch) {
    return V >= 1 && V <= (1 << 21) && n >= 1 && n <= kMaxDrafts && batch >= 0;
}

int check_solve_args(const void* q_logits, const void* p_logits, int dtype, int V, int n, int topk, float temp_target,
                     float temp_draft, int batch, const gr_options* opt, const void* params, const float* alpha_star,
                     const int* status, SolveSetup* out)
{
    if (!shape_ok(V, n, batch)) return GR_E_INVALID;
    if (dtype != GR_F32 && dtype != GR_BF16) return GR_E_INVALID;
    if (!(temp_target > 0.f) || !(temp_draft > 0.f) || !isfinite(temp_target) || !isfinite(temp_draft))
        return GR_E_INVALID;
    out->tol = 3e-7; out->qstep = 0.4; out->max_iters = 40; out->tau = 0.0;
    out->scan_done = nullptr; out->force_robust = 0;
    if (opt) {
        out->scan_done = (cudaEvent_t)opt->scan_done_event;
        out->force_robust = opt->force_robust;
        out->tol = opt->tol; out->max_iters = opt->max_iters; out->qstep = opt->quad_step; out->tau = opt->tau;
        if (!(out->tol > 0.0) || out->max_iters < 1 || !(out->qstep >= 0.05 && out->qstep <= 2.0)) return GR_E_INVALID;
        if (!(out->tau >= 0.0) || !(out->tau <= 1.0)) return GR_E_INVALID;
    }
    out->kfull = (topk <= 0 || topk >= V) ? V : topk;
    out->kcap = kcap_of(V, topk);
    out->pstride = params_stride(V, topk);
    if (batch == 0) return GR_OK;
    if (!q_logits || !p_logits || !params || !alpha_star || !status) return GR_E_NULL;
    if (((uintptr_t)q_logits & 15) || ((uintptr_t)p_logits & 15) || ((uintptr_t)params & 15)) return GR_E_ALIGN;
    if (out->kcap == 0 && out->kfull != V) return GR_E_TOO_LARGE;   // a truncated support beyond the capacity
    return GR_OK;
}
}  // namespace gr

extern "C" {

size_t gr_params_bytes(int V, int n, int topk, int batch)
{
    if (!gr::shape_ok(V, n, batch)) return 0;
    size_t s = (size_t)gr::params_stride(V, topk) * (size_t)(batch > 0 ? batch : 1);
    return s;
}

size_t gr_workspace_bytes(int V, int n, int topk, int batch)
{
    if (!gr::shape_ok(V, n, batch)) return 0;
    const size_t nb = (size_t)(batch > 0 ? batch : 1);
    size_t s = (size_t)gr::ws_stride() * nb;
    // an untruncated draft on a vocabulary beyond the solve capacity: room to sort the row for alpha*
    if (gr::kcap_of(V, topk) == 0) s += gr::fullsort_scratch_bytes(V) * nb;
    return s;
}

static int solve_impl(const void* q_logits, const void* p_logits, int dtype, int V, int n, int topk, float temp_target,
                      float temp_draft, int batch, const gr_options* opt, void* params, void* workspace,
                      float* alpha_star, int* status, gr::FusedArgs fa, void* stream)
{
    gr::SolveSetup su;
    const int chk = gr::check_solve_args(q_logits, p_logits, dtype, V, n, topk, temp_target, temp_draft, batch, opt,
                                         params, alpha_star, status, &su);
    if (chk != GR_OK) return chk;
    if (batch == 0) return GR_OK;
    if (!workspace) return GR_E_NULL;
    if ((uintptr_t)workspace & 15) return GR_E_ALIGN;
    const double tol = su.tol, qstep = su.qstep, tau = su.tau;
    const int max_iters = su.max_iters, force_robust = su.force_robust;
    cudaEvent_t scan_done = su.scan_done;
    const int kfull = su.kfull, kcap = su.kcap, pstride = su.pstride;
    const bool full_large = kcap == 0;
    cudaStream_t st = (cudaStream_t)stream;
    gr::NvtxRange whole(fa.draft ? "gr_solve_verify" : "gr_solve");
    {
        gr::NvtxRange r("gr:scan");
        gr::launch_scan(q_logits, p_logits, dtype, V, kfull, full_large, (double)temp_target, (double)temp_draft,
                        batch, (char*)workspace, (char*)params, pstride, kcap, st);
    }
    if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return GR_E_LAUNCH; }
    if (scan_done && cudaEventRecord(scan_done, st) != cudaSuccess) { cudaGetLastError(); return GR_E_LAUNCH; }
    gr::NvtxRange r(fa.draft ? "gr:solve+draw" : "gr:solve");
    int rc = gr::launch_solve_any((const char*)workspace, (char*)params, pstride, kcap, V, n, topk,
                                  (double)temp_target, (double)temp_draft, tol, max_iters, qstep, tau, batch,
                                  force_robust, alpha_star, status, fa, st);
    if (rc != GR_OK) return rc;
    if (full_large) {
        // no rule is solved for this shape, but the optimal acceptance still is (bucketed search for the minimum of
        // psi, or with force_robust a sort of the whole row and a prefix scan)
        char* scratch = (char*)workspace + (size_t)gr::ws_stride() * (size_t)batch;
        gr::launch_fullsort(q_logits, p_logits, dtype, V, n, (double)temp_target, (double)temp_draft, batch,
                            (const char*)workspace, scratch, (char*)params, pstride, force_robust, alpha_star, 1, 0,
                            nullptr, st);
    }
    if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return GR_E_LAUNCH; }
    return GR_OK;
}

int gr_solve(const void* q_logits, const void* p_logits, int dtype, int V, int n, int topk, float temp_target,
             float temp_draft, int batch, const gr_options* opt, void* params, void* workspace, float* alpha_star,
             int* status, void* stream)
{
    gr::FusedArgs none = {nullptr, nullptr, nullptr, nullptr, nullptr};
    return solve_impl(q_logits, p_logits, dtype, V, n, topk, temp_target, temp_draft, batch, opt, params, workspace,
                      alpha_star, status, none, stream);
}

int gr_solve_verify(const void* q_logits, const void* p_logits, int dtype, int V, int n, int topk, float temp_target,
                    float temp_draft, int batch, const gr_options* opt, const int* draft_tokens, const float* uniforms,
                    void* params, void* workspace, float* alpha_star, int* out_token, unsigned char* out_accepted,
                    int* status, void* stream)
{
    if (batch > 0 && (!draft_tokens || !uniforms || !out_token || !out_accepted)) return GR_E_NULL;
    gr::FusedArgs fa = {draft_tokens, uniforms, out_token, out_accepted, status};
    return solve_impl(q_logits, p_logits, dtype, V, n, topk, temp_target, temp_draft, batch, opt, params, workspace,
                      alpha_star, status, fa, stream);
}

int gr_alpha_star(const void* q_logits, const void* p_logits, int dtype, int V, const int* n_list, int n_count,
                  int topk, float temp_target, float temp_draft, int batch, void* workspace, float* alpha_star,
                  int* status, void* stream)
{
    if (!gr::shape_ok(V, 1, batch)) return GR_E_INVALID;
    if (dtype != GR_F32 && dtype != GR_BF16) return GR_E_INVALID;
    if (!(temp_target > 0.f) || !(temp_draft > 0.f) || !isfinite(temp_target) || !isfinite(temp_draft))
        return GR_E_INVALID;
    if (!n_list) return GR_E_NULL;
    if (n_count < 1 || n_count > GR_MAX_ALPHA_N) return GR_E_INVALID;
    for (int i = 0; i < n_count; i++)
        if (n_list[i] < 1 || n_list[i] > gr::kMaxDrafts) return GR_E_INVALID;
    if (batch == 0) return GR_OK;
    if (!q_logits || !p_logits || !workspace || !alpha_star || !status) return GR_E_NULL;
    if (((uintptr_t)q_logits & 15) || ((uintptr_t)p_logits & 15) || ((uintptr_t)workspace & 15)) return GR_E_ALIGN;
    const int kfull = (topk <= 0 || topk >= V) ? V : topk;
    const int kcap = gr::kcap_of(V, topk);
    if (kcap == 0 && kfull != V) return GR_E_TOO_LARGE;       // a truncated support beyond the capacity
    cudaStream_t st = (cudaStream_t)stream;
    gr::NvtxRange whole("gr_alpha_star");
    if (kcap == 0) {
        // untruncated draft on a large vocabulary: the streaming pass for the row statistics, then the bucketed
        // search for min psi once per draft count (rows it cannot separate take the sort)
        gr::launch_scan(q_logits, p_logits, dtype, V, kfull, true, (double)temp_target, (double)temp_draft, batch,
                        (char*)workspace, nullptr, 0, kcap, st);
        char* scratch = (char*)workspace + (size_t)gr::ws_stride() * (size_t)batch;
        for (int j = 0; j < n_count; j++)
            gr::launch_fullsort(q_logits, p_logits, dtype, V, n_list[j], (double)temp_target, (double)temp_draft, batch,
                                (const char*)workspace, scratch, nullptr, 0, 0, alpha_star, n_count, j, status, st);
        if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return GR_E_LAUNCH; }
        return GR_OK;
    }
    gr::launch_scan(q_logits, p_logits, dtype, V, kfull, false, (double)temp_target, (double)temp_draft, batch,
                    (char*)workspace, nullptr, 0, kcap, st);
    gr::launch_alpha((const char*)workspace, V, topk, (double)temp_target, (double)temp_draft, n_list, n_count, batch,
                     alpha_star, status, st);
    if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return GR_E_LAUNCH; }
    return GR_OK;
}

int gr_verify(const void* params, const int* draft_tokens, const float* uniforms, int batch, int* out_token,
              unsigned char* out_accepted, int* status, void* stream)
{
    if (batch < 0) return GR_E_INVALID;
    if (batch == 0) return GR_OK;
    if (!params || !draft_tokens || !uniforms || !out_token || !out_accepted || !status) return GR_E_NULL;
    if ((uintptr_t)params & 15) return GR_E_ALIGN;
    gr::NvtxRange whole("gr_verify");
    gr::launch_verify((const char*)params, draft_tokens, uniforms, batch, out_token, out_accepted, status,
                      (cudaStream_t)stream);
    if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return GR_E_LAUNCH; }
    return GR_OK;
}

int gr_read_rule(const void* params, int batch, int kcap, int* ids, int* block, double* w, double* resid,
                 double* flow, double* header, void* stream)
{
    if (batch < 0 || kcap < 0) return GR_E_INVALID;
    if (batch == 0) return GR_OK;
    if (!params) return GR_E_NULL;
    gr::launch_read_rule((const char*)params, batch, kcap, ids, block, w, resid, flow, header, (cudaStream_t)stream);
    if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return GR_E_LAUNCH; }
    return GR_OK;
}

int gr_read_slice(const void* params, const int* draft_tokens, int batch, int n, int* U, double* pi, double* rho,
                  int* status, void* stream)
{
    if (batch < 0 || n < 1 || n > gr::kMaxDrafts) return GR_E_INVALID;
    if (batch == 0) return GR_OK;
    if (!params || !draft_tokens || !U || !pi || !rho || !status) return GR_E_NULL;
    if ((uintptr_t)params & 15) return GR_E_ALIGN;
    gr::launch_read_slice((const char*)params, draft_tokens, batch, n, U, pi, rho, status, (cudaStream_t)stream);
    if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return GR_E_LAUNCH; }
    return GR_OK;
}

#ifdef GR_CHECK
// Bounds-checked build only: exercises the checked pointer itself.  A kernel reads and writes a 4-entry shared
// array through it at indices -1 .. 4; out[0] = number of accesses that were skipped and flagged (expected 2),
// out[1] = sum of what the in-range reads returned (expected 0+1+2+3), out[2] = the values the skipped reads gave.
namespace gr {
__global__ void check_selftest_kernel(int* out)
{
    __shared__ int arr[4];
    __shared__ int flag;
    if (threadIdx.x == 0) {
        for (int i = 0; i < 4; i++) arr[i] = i;
        int skipped = 0, sum = 0, ghost = 0;
        for (int i = -1; i <= 4; i++) {
            flag = 0;
            CkPtr<int> p(arr, 4, &flag);
            const int v = p[i];
            p[i] = v;                       // a skipped write must not land anywhere
            if (flag) { skipped++; ghost += v; } else sum += v;
        }
        out[0] = skipped; out[1] = sum; out[2] = ghost;
        out[3] = arr[0] + arr[1] + arr[2] + arr[3];
    }
}
}  // namespace gr
int gr_check_selftest(int* out_device, void* stream)
{
    gr::check_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(out_device);
    return cudaPeekAtLastError() == cudaSuccess ? GR_OK : GR_E_LAUNCH;
}
#endif

const char* gr_strerror(int code)
{
    switch (code) {
        case GR_OK: return "ok";
        case GR_NOT_CONVERGED: return "iteration cap reached before the gradient tolerance";
        case GR_SUPPORT_TOO_LARGE: return "draft support larger than GR_MAX_SUPPORT: rule not solved";
        case GR_BAD_LOGITS: return "NaN or infinite logit";
        case GR_DRAFT_OUT_OF_SUPPORT: return "drafted token outside the draft support";
        case GR_STALE_PARAMS: return "params block was not written by gr_solve";
        case GR_PARTIAL_RULE: return "rule solved only for the drafts given to gr_solve_verify";
        case GR_CHECK_FAILED: return "bounds-checked build: an out-of-range access was skipped";
        case GR_E_INVALID: return "invalid size, temperature or option";
        case GR_E_NULL: return "required pointer is NULL";
        case GR_E_ALIGN: return "pointer is not 16-byte aligned";
        case GR_E_LAUNCH: return "CUDA launch failed";
        case GR_E_TOO_LARGE: return "shape beyond the library's capacity";
        default: return "unknown code";
    }
}

}  // extern "C"
