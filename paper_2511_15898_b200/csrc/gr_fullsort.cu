// Optimal acceptance for an untruncated draft on a large vocabulary (support = V > GR_MAX_SUPPORT).
//
// The rule itself is not solved there (status GR_SUPPORT_TOO_LARGE), but alpha* = 1 + min_H psi(H) only needs
// the ratio order of the whole vocabulary and a prefix scan (Eq. "subset-select", Sec. 5.1): one CTA per
// instance sorts (log-ratio key, id) pairs of the row in global scratch with a bitonic network, then scans
// tgt and drf along the order and takes the minimum of psi_j = Tg_j - Dr_j^n.
// The network's passes with a compare distance below the tile size (4096 pairs, 48 KB) run on tiles staged in
// shared memory: 15 trips through global memory for a 65536-entry row instead of 136.
#include "gr_common.cuh"

namespace gr {

constexpr int kFsThreads = 1024;
constexpr int kFsTile = 4096;          // pairs per shared-memory tile
constexpr int kFsSmemBytes = kFsTile * 12;

__host__ __device__ inline int next_pow2(int v) { int p = 1; while (p < v) p <<= 1; return p; }
__host__ size_t fullsort_scratch_bytes(int V) { return (size_t)next_pow2(V) * 12; }

// order-preserving map double -> uint64 (larger double, larger key)
__device__ inline unsigned long long dkey(double x) {
    unsigned long long u = (unsigned long long)__double_as_longlong(x);
    return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}
// true when (ka, ia) comes before (kb, ib): larger key first, equal keys by smaller id
__device__ inline bool before(unsigned long long ka, int ia, unsigned long long kb, int ib) {
    return ka > kb || (ka == kb && ia < ib);
}

template <typename T>
__global__ void __launch_bounds__(kFsThreads)
fullsort_alpha_kernel(const T* __restrict__ q, const T* __restrict__ p, int V, int n, double temp_t, double temp_d,
                      const char* __restrict__ ws, char* __restrict__ scratch, char* __restrict__ params, int pstride,
                      float* __restrict__ alpha_out)
{
    __shared__ double s_a[kFsThreads / 32], s_b[kFsThreads / 32];
    __shared__ double s_carry[2];
    __shared__ double s_min[kFsThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long b = blockIdx.x;
    const WsHeader* wh = reinterpret_cast<const WsHeader*>(ws + (size_t)b * ws_stride());
    Header* hdr = reinterpret_cast<Header*>(params + (size_t)b * pstride);
    if (wh->bad != 0) return;                       // header already says GR_BAD_LOGITS
    const T* qrow = q + (size_t)b * V;
    const T* prow = p + (size_t)b * V;
    const int VP = next_pow2(V);
    unsigned long long* key = reinterpret_cast<unsigned long long*>(scratch + (size_t)b * VP * 12);
    int* idx = reinterpret_cast<int*>(key + VP);
    for (int i = tid; i < VP; i += kFsThreads) {
        if (i < V) {
            const double a = (double)load_logit<T>(qrow, i) / temp_t;
            const double d = (double)load_logit<T>(prow, i) / temp_d;
            key[i] = dkey(d - a); idx[i] = i;
        } else {
            key[i] = 0ull; idx[i] = 0x7fffffff;     // padding sorts last
        }
    }
    __syncthreads();
    // bitonic network over the VP pairs ("before" order ascending in position).  Compare-exchange of positions
    // i < l in the stage of block size k: ascending when (i & k) == 0.
    extern __shared__ __align__(16) unsigned char fs_smem[];
    unsigned long long* tk = reinterpret_cast<unsigned long long*>(fs_smem);
    int* ti = reinterpret_cast<int*>(tk + kFsTile);
    const int TL = VP < kFsTile ? VP : kFsTile;
    // the passes of distance j0, j0/2, ..., 1 of stage k on every tile, in shared memory; with whole = true all
    // stages 2 .. TL of the tile (the network's first log2 TL stages)
    auto tile_passes = [&](int k, int j0, bool whole) {
        for (int t0 = 0; t0 < VP; t0 += TL) {
            for (int e = tid; e < TL; e += kFsThreads) { tk[e] = key[t0 + e]; ti[e] = idx[t0 + e]; }
            __syncthreads();
            for (int kk = whole ? 2 : k; kk <= (whole ? TL : k); kk <<= 1) {
                for (int j2 = whole ? (kk >> 1) : j0; j2 > 0; j2 >>= 1) {
                    for (int pr = tid; pr < TL / 2; pr += kFsThreads) {
                        const int i = 2 * pr - (pr & (j2 - 1)), l = i + j2;
                        const unsigned long long ki = tk[i], kl = tk[l];
                        const int ii = ti[i], il = ti[l];
                        const bool up = ((t0 + i) & kk) == 0;
                        const bool wrong = up ? before(kl, il, ki, ii) : before(ki, ii, kl, il);
                        if (wrong) { tk[i] = kl; tk[l] = ki; ti[i] = il; ti[l] = ii; }
                    }
                    __syncthreads();
                }
            }
            for (int e = tid; e < TL; e += kFsThreads) { key[t0 + e] = tk[e]; idx[t0 + e] = ti[e]; }
            __syncthreads();
        }
    };
    tile_passes(0, 0, true);
    for (int k = 2 * TL; k <= VP; k <<= 1) {
        for (int j2 = k >> 1; j2 >= TL; j2 >>= 1) {
            for (int pr = tid; pr < VP / 2; pr += kFsThreads) {
                const int i = 2 * pr - (pr & (j2 - 1)), l = i + j2;
                const unsigned long long ki = key[i], kl = key[l];
                const int ii = idx[i], il = idx[l];
                const bool up = (i & k) == 0;
                const bool wrong = up ? before(kl, il, ki, ii) : before(ki, ii, kl, il);
                if (wrong) { key[i] = kl; key[l] = ki; idx[i] = il; idx[l] = ii; }
            }
            __syncthreads();
        }
        tile_passes(k, TL >> 1, false);
    }
    // log-sum-exp of both rows in fp64 (the streaming kernel's fp32 sums are good to ~1e-7 only, and the draft's
    // error enters alpha* multiplied by n through Dr^n)
    double mt = -1.0e300, md = -1.0e300;
    for (int i = tid; i < V; i += kFsThreads) {
        mt = fmax(mt, (double)load_logit<T>(qrow, i) / temp_t);
        md = fmax(md, (double)load_logit<T>(prow, i) / temp_d);
    }
    for (int o = 16; o > 0; o >>= 1) {
        mt = fmax(mt, __shfl_xor_sync(0xffffffffu, mt, o));
        md = fmax(md, __shfl_xor_sync(0xffffffffu, md, o));
    }
    if (lane == 0) { s_a[warp] = mt; s_b[warp] = md; }
    __syncthreads();
    mt = s_a[0]; md = s_b[0];
    for (int w2 = 1; w2 < kFsThreads / 32; w2++) { mt = fmax(mt, s_a[w2]); md = fmax(md, s_b[w2]); }
    __syncthreads();
    double st0 = 0.0, sd0 = 0.0;
    for (int i = tid; i < V; i += kFsThreads) {
        st0 += exp((double)load_logit<T>(qrow, i) / temp_t - mt);
        sd0 += exp((double)load_logit<T>(prow, i) / temp_d - md);
    }
    for (int o = 16; o > 0; o >>= 1) {
        st0 += __shfl_xor_sync(0xffffffffu, st0, o);
        sd0 += __shfl_xor_sync(0xffffffffu, sd0, o);
    }
    if (lane == 0) { s_a[warp] = st0; s_b[warp] = sd0; }
    __syncthreads();
    st0 = 0.0; sd0 = 0.0;
    for (int w2 = 0; w2 < kFsThreads / 32; w2++) { st0 += s_a[w2]; sd0 += s_b[w2]; }
    __syncthreads();
    const double lse_t = mt + log(st0), lse_d = md + log(sd0);
    // prefix sums of tgt and drf along the order, psi_j = Tg_j - Dr_j^n, running minimum
    if (tid == 0) { s_carry[0] = 0.0; s_carry[1] = 0.0; }
    __syncthreads();
    double best = 0.0;                              // psi of the empty prefix
    constexpr int kPer = 4;
    for (int base = 0; base < V; base += kFsThreads * kPer) {
        double ta[kPer], da[kPer];
        double st = 0.0, sd = 0.0;
#pragma unroll
        for (int u = 0; u < kPer; u++) {
            const int j = base + tid * kPer + u;
            double tv = 0.0, dv = 0.0;
            if (j < V) {
                const int id = idx[j];
                tv = exp((double)load_logit<T>(qrow, id) / temp_t - lse_t);
                dv = exp((double)load_logit<T>(prow, id) / temp_d - lse_d);
            }
            st += tv; sd += dv; ta[u] = st; da[u] = sd;
        }
        // exclusive offsets of this thread: warp scan, then across warps
        double wt = st, wd = sd;
        for (int o = 1; o < 32; o <<= 1) {
            const double t2 = __shfl_up_sync(0xffffffffu, wt, o), d2 = __shfl_up_sync(0xffffffffu, wd, o);
            if (lane >= o) { wt += t2; wd += d2; }
        }
        if (lane == 31) { s_a[warp] = wt; s_b[warp] = wd; }
        __syncthreads();
        double ot = s_carry[0], od = s_carry[1];
        for (int w2 = 0; w2 < warp; w2++) { ot += s_a[w2]; od += s_b[w2]; }
        ot += wt - st; od += wd - sd;
#pragma unroll
        for (int u = 0; u < kPer; u++) {
            const int j = base + tid * kPer + u;
            if (j < V) {
                double Tg = ot + ta[u], Dr = od + da[u];
                if (j == V - 1) { Tg = 1.0; Dr = 1.0; }     // both distributions are normalised
                const double psi = Tg - pow(Dr, (double)n);
                best = fmin(best, psi);
            }
        }
        __syncthreads();
        if (tid == kFsThreads - 1) { s_carry[0] = ot + st; s_carry[1] = od + sd; }
        __syncthreads();
    }
    for (int o = 16; o > 0; o >>= 1) best = fmin(best, __shfl_xor_sync(0xffffffffu, best, o));
    if (lane == 0) s_min[warp] = best;
    __syncthreads();
    if (tid == 0) {
        for (int w2 = 1; w2 < kFsThreads / 32; w2++) best = fmin(best, s_min[w2]);
        hdr->alpha_star = 1.0 + best;
        hdr->resid_total = -best;
        alpha_out[b] = (float)(1.0 + best);
    }
}

void launch_fullsort(const void* q, const void* p, int dtype, int V, int n, double temp_t, double temp_d, int batch,
                     const char* ws, char* scratch, char* params, int pstride, float* alpha_out, cudaStream_t st)
{
    // function attributes belong to the device: set once per device (a failure shows up as a launch error)
    static bool configured[kMaxDevices] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) dev = -1;
    if (dev < 0 || !configured[dev]) {
        const bool ok = cudaFuncSetAttribute(fullsort_alpha_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kFsSmemBytes) == cudaSuccess &&
                        cudaFuncSetAttribute(fullsort_alpha_kernel<__nv_bfloat16>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, kFsSmemBytes) == cudaSuccess;
        if (dev >= 0 && ok) configured[dev] = true;
    }
    if (dtype == GR_F32)
        fullsort_alpha_kernel<float><<<batch, kFsThreads, kFsSmemBytes, st>>>((const float*)q, (const float*)p, V, n, temp_t,
                                                                   temp_d, ws, scratch, params, pstride, alpha_out);
    else
        fullsort_alpha_kernel<__nv_bfloat16><<<batch, kFsThreads, kFsSmemBytes, st>>>((const __nv_bfloat16*)q,
                                                                           (const __nv_bfloat16*)p, V, n, temp_t,
                                                                           temp_d, ws, scratch, params, pstride,
                                                                           alpha_out);
}

}  // namespace gr
