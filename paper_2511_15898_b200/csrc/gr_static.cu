// gr_solve_static: gr_solve for callers that may not allocate device memory.
//
// The scratch that gr_solve takes as its `workspace` argument lives here in a
// file-scope device array instead, so the caller passes inputs and outputs only.
#include "gr_host.h"

namespace gr {
constexpr int kStaticBytes = GR_STATIC_MAX_BATCH * (int)(sizeof(WsHeader) + kMaxSupport * 12);

// Every GPU that loads the library holds this array (about 0.4 MB) until the process exits.
static __device__ __align__(256) unsigned char g_static_workspace[kStaticBytes];

// The array's name is only a host-side handle in host code; the address a kernel can use is
// asked for once per device, with that device current, and remembered.
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
    gr::SolveSetup su;
    const int chk = gr::check_solve_args(q_logits, p_logits, dtype, V, n, topk, temp_target, temp_draft, batch, opt,
                                         params, alpha_star, status, &su);
    if (chk != GR_OK) return chk;
    if (batch > GR_STATIC_MAX_BATCH) return GR_E_TOO_LARGE;      // the built-in scratch holds this many instances
    if (batch == 0) return GR_OK;
    const double tol = su.tol, qstep = su.qstep, tau = su.tau;
    const int max_iters = su.max_iters, force_robust = su.force_robust;
    cudaEvent_t scan_done = su.scan_done;
    const int kfull = su.kfull, kcap = su.kcap;
    const bool full_large = kcap == 0;
    if (full_large) return GR_E_TOO_LARGE;     // (the built-in scratch has no room for the whole-vocabulary sort)
    char* ws = nullptr;
    const int rs = gr::static_workspace(&ws);
    if (rs != GR_OK) return rs;
    const int pstride = su.pstride;
    cudaStream_t st = (cudaStream_t)stream;
    gr::NvtxRange whole("gr_solve_static");
    // the streaming kernel writes every workspace field the solve kernel reads, so nothing has to be cleared
    gr::launch_scan(q_logits, p_logits, dtype, V, kfull, full_large, (double)temp_target, (double)temp_draft, batch,
                    ws, (char*)params, pstride, kcap, st);
    if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return GR_E_LAUNCH; }
    if (scan_done && cudaEventRecord(scan_done, st) != cudaSuccess) { cudaGetLastError(); return GR_E_LAUNCH; }
    const int rc = gr::launch_solve_any(ws, (char*)params, pstride, kcap, V, n, topk, (double)temp_target,
                                        (double)temp_draft, tol, max_iters, qstep, tau, batch, force_robust, alpha_star,
                                        status, gr::FusedArgs{nullptr, nullptr, nullptr, nullptr, nullptr}, st);
    if (rc != GR_OK) return rc;
    if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return GR_E_LAUNCH; }
    return GR_OK;
}
