// Dispatch of the fast per-instance solve (kernels in gr_fast.cuh; one translation unit per series length and
// padded support size).
#include "gr_verify.cuh"

namespace gr {

#define GR_FAST_ARGS                                                                                              \
    const char *ws, char *params, int pstride, int kcap, int V, int n, int topk, double temp_t, double temp_d,   \
        double tol, int max_iters, double qstep, double tau, int batch, float *alpha_out, int *status_out,       \
        FusedArgs fa, cudaStream_t st
namespace fast64 {
int launch_fast_n4(GR_FAST_ARGS);
int launch_fast_n8(GR_FAST_ARGS);
int launch_fast_n16(GR_FAST_ARGS);
}
namespace fast128 {
int launch_fast_n8(GR_FAST_ARGS);
int launch_fast_n16(GR_FAST_ARGS);
}

// Returns 1 when no fast variant covers the shape (the caller then runs the robust kernel on everything);
// after a return of 0 the caller runs the robust kernel on the instances this one flagged (normally none).
int launch_fast(GR_FAST_ARGS)
{
    if (kcap <= 0 || kcap > 128 || n > 16 || n < 2) return 1;
#define GR_FAST_PASS ws, params, pstride, kcap, V, n, topk, temp_t, temp_d, tol, max_iters, qstep, tau, batch, alpha_out, status_out, fa, st
    if (kcap <= 64) {
        if (n <= 4) return fast64::launch_fast_n4(GR_FAST_PASS);
        if (n <= 8) return fast64::launch_fast_n8(GR_FAST_PASS);
        return fast64::launch_fast_n16(GR_FAST_PASS);
    }
    if (n <= 8) return fast128::launch_fast_n8(GR_FAST_PASS);
    return fast128::launch_fast_n16(GR_FAST_PASS);
}

}  // namespace gr
