// Host-side declarations shared by the translation units that implement the C interface: the kernel launchers and
// the argument checks common to gr_solve, gr_solve_verify and gr_solve_static.
#pragma once
#include <nvtx3/nvToolsExt.h>
#include "gr_verify.cuh"

namespace gr {

// A named range on a profiler's timeline around the host code that enqueues one phase of the path (scan, solve,
// verify ...).  Without a profiler attached the two calls do nothing.
struct NvtxRange {
    explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
    NvtxRange(const NvtxRange&) = delete;
    NvtxRange& operator=(const NvtxRange&) = delete;
};

void launch_scan(const void* q, const void* p, int dtype, int V, int ksel, bool full_large, double temp_t,
                 double temp_d, int batch, char* ws, char* params, int pstride, int kcap, cudaStream_t st);
int launch_solve(const char* ws, char* params, int pstride, int kcap, int V, int n, int topk, double temp_t,
                 double temp_d, double tol, int max_iters, double qstep, double tau, int batch, int only_flagged,
                 float* alpha_out, int* status_out, FusedArgs fa, cudaStream_t st);
int launch_fast(const char* ws, char* params, int pstride, int kcap, int V, int n, int topk, double temp_t,
                double temp_d, double tol, int max_iters, double qstep, double tau, int batch, float* alpha_out,
                int* status_out, FusedArgs fa, cudaStream_t st);
int launch_solve_any(const char* ws, char* params, int pstride, int kcap, int V, int n, int topk, double temp_t,
                     double temp_d, double tol, int max_iters, double qstep, double tau, int batch, int force_robust,
                     float* alpha_out, int* status_out, FusedArgs fa, cudaStream_t st);
size_t fullsort_scratch_bytes(int V);
void launch_fullsort(const void* q, const void* p, int dtype, int V, int n, double temp_t, double temp_d, int batch,
                     const char* ws, char* scratch, char* params, int pstride, int force_sort, float* alpha_out,
                     int out_stride, int out_off, int* status_out, cudaStream_t st);
void launch_alpha(const char* ws, int V, int topk, double temp_t, double temp_d, const int* n_list, int n_count,
                  int batch, float* alpha_out, int* status_out, cudaStream_t st);
void launch_verify(const char* params, const int* draft, const float* uni, int batch, int* out_token,
                   unsigned char* out_acc, int* status, cudaStream_t st);
void launch_read_slice(const char* params, const int* draft, int batch, int n, int* U, double* pi, double* rho,
                       int* status, cudaStream_t st);
void launch_read_rule(const char* params, int batch, int kcap, int* ids, int* block, double* w, double* resid,
                      double* flow, double* header, cudaStream_t st);

// The solver options after defaults and range checks.
struct SolveSetup {
    double tol, qstep, tau;
    int max_iters, force_robust;
    cudaEvent_t scan_done;
    int kfull, kcap, pstride;      // support size asked for, capacity of the per-support arrays (0: beyond it), params stride
};

// Checks shared by the solving entry points (everything but the workspace pointer, which only some of them take).
// Returns GR_OK or the GR_E_* code to hand back; fills `out` on GR_OK.
int check_solve_args(const void* q_logits, const void* p_logits, int dtype, int V, int n, int topk, float temp_target,
                     float temp_draft, int batch, const gr_options* opt, const void* params, const float* alpha_star,
                     const int* status, SolveSetup* out);

}  // namespace gr
