// gr_solve_static: gr_solve for callers that may not allocate device memory.
//
// The scratch that gr_solve takes as its `workspace` argument lives here in a
// file-scope device array instead, so the caller passes inputs and outputs only.
#include <math.h>
#include "gr_verify.cuh"

namespace gr {
void launch_scan(const void* q, const void* p, int dtype, int V, int ksel, bool full_large, double temp_t,
                 double temp_d, int batch, char* ws, char* params, int pstride, int kcap, cudaStream_t st);
int launch_solve_any(const char* ws, char* params, int pstride, int kcap, int V, int n, int topk, double temp_t,
                     double temp_d, double tol, int max_iters, double qstep, int batch, int force_robust,
                     float* alpha_out, int* status_out, FusedArgs fa, cudaStream_t st);

constexpr int kStaticBytes = GR_STATIC_MAX_BATCH * (int)(sizeof(WsHeader) + kMaxSupport * 12);

// Every GPU that loads the library holds this array (about 0.4 MB) until the process exits.
static __device__ __align__(256) unsigned char g_static_workspace[kStaticBytes];

// The array's name is only a host-side handle in host code; the address a kernel can use is
// asked for once per device, with that device current, and remembered.
constexpr int kMaxDevices = 64;
static char* g_static_ptr[kMaxDevices] = {nullptr};

static int static_workspace(char** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return GR_E_LAUNCH; }
    if (g_static_ptr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_workspace) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return GR_E_LAUNCH;
        }
        g_static_ptr[dev] = (char*)ptr;
    }
    *out = g_static_ptr[dev];
    return GR_OK;
}
}  // namespace gr

extern "C" int gr_solve_static(const void* q_logits, const void* p_logits, int dtype, int V, int n, int topk,
                               float temp_target, float temp_draft, int batch, const gr_options* opt, void* params,
                               float* alpha_star, int* status, void* stream)
{
    if (!(V >= 1 && V <= (1 << 21) && n >= 1 && n <= gr::kMaxDrafts && batch >= 0)) return GR_E_INVALID;
    if (batch > GR_STATIC_MAX_BATCH) return GR_E_TOO_LARGE;      // the built-in scratch holds this many instances
    if (dtype != GR_F32 && dtype != GR_BF16) return GR_E_INVALID;
    if (!(temp_target > 0.f) || !(temp_draft > 0.f) || !isfinite(temp_target) || !isfinite(temp_draft))
        return GR_E_INVALID;
    double tol = 1e-9, qstep = 0.4;
    int max_iters = 40;
    cudaEvent_t scan_done = nullptr;
    int force_robust = 0;
    if (opt) {
        scan_done = (cudaEvent_t)opt->scan_done_event;
        force_robust = opt->force_robust;
        tol = opt->tol; max_iters = opt->max_iters; qstep = opt->quad_step;
        if (!(tol > 0.0) || max_iters < 1 || !(qstep >= 0.05 && qstep <= 2.0)) return GR_E_INVALID;
    }
    if (batch == 0) return GR_OK;
    if (!q_logits || !p_logits || !params || !alpha_star || !status) return GR_E_NULL;
    if (((uintptr_t)q_logits & 15) || ((uintptr_t)p_logits & 15) || ((uintptr_t)params & 15)) return GR_E_ALIGN;
    const int kfull = (topk <= 0 || topk >= V) ? V : topk;
    const int kcap = gr::kcap_of(V, topk);
    const bool full_large = kcap == 0;
    if (full_large) return GR_E_TOO_LARGE;     // (the built-in scratch has no room for the whole-vocabulary sort)
    char* ws = nullptr;
    const int rs = gr::static_workspace(&ws);
    if (rs != GR_OK) return rs;
    const int pstride = gr::params_stride(V, topk);
    cudaStream_t st = (cudaStream_t)stream;
    // the streaming kernel writes every workspace field the solve kernel reads, so nothing has to be cleared
    gr::launch_scan(q_logits, p_logits, dtype, V, kfull, full_large, (double)temp_target, (double)temp_draft, batch,
                    ws, (char*)params, pstride, kcap, st);
    if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return GR_E_LAUNCH; }
    if (scan_done && cudaEventRecord(scan_done, st) != cudaSuccess) { cudaGetLastError(); return GR_E_LAUNCH; }
    const int rc = gr::launch_solve_any(ws, (char*)params, pstride, kcap, V, n, topk, (double)temp_target,
                                        (double)temp_draft, tol, max_iters, qstep, batch, force_robust, alpha_star,
                                        status, gr::FusedArgs{nullptr, nullptr, nullptr, nullptr, nullptr}, st);
    if (rc != GR_OK) return rc;
    if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return GR_E_LAUNCH; }
    return GR_OK;
}
