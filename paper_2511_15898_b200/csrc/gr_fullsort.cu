// Optimal acceptance for an untruncated draft on a large vocabulary (support = V > GR_MAX_SUPPORT).
//
// The rule itself is not solved there (status GR_SUPPORT_TOO_LARGE), but alpha* = 1 + min_H psi(H) only needs
// the ratio order of the whole vocabulary and a prefix scan (Eq. "subset-select", Sec. 5.1):
// psi_j = Tg_j - Dr_j^n over the prefixes of the order by descending draft / target ratio.
//
// bucket_alpha_kernel finds that minimum without sorting the row: the log-ratio keys are binned into 4096 equal
// buckets (a monotone map, so the bucket order is the ratio order), the bucket masses give psi exactly at every
// bucket boundary, and a lower bound on psi inside a bucket (the ratios inside it span one bucket width) leaves
// only the few buckets next to the minimum to be ordered exactly, in shared memory.  Three passes over the row.
// A row whose candidate buckets do not fit is handed to fullsort_alpha_kernel: one CTA per instance sorts (key, id)
// pairs of the row in global scratch with a bitonic network, then scans tgt and drf along the order.
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

constexpr int kBkThreads = 1024;
constexpr int kBkBuckets = 4096;
constexpr int kBkPer = kBkBuckets / kBkThreads;   // buckets per thread in the scan over buckets
constexpr int kBkMaxCand = 4096;                  // elements of candidate buckets held in shared memory
constexpr int kBkMaxPerBucket = 256;              // largest candidate bucket ordered in shared memory
constexpr double kBkScale = 4398046511104.0;      // 2^42: masses are summed as integers (exact, order-free)
constexpr int kBkSmemBytes = kBkBuckets * (8 + 8 + 4 + 4) + kBkMaxCand * (8 + 4 + 4);

__device__ inline unsigned long long mass_fixed(double x, double mx) { return (unsigned long long)llrint(exp(x - mx) * kBkScale); }

// Exclusive prefix over the CTA of one 64-bit integer per thread; *total gets the sum.  s_w: kBkThreads / 32 slots.
__device__ inline unsigned long long block_exscan_u64(unsigned long long v, unsigned long long* s_w,
                                                      unsigned long long* total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long inc = v;
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();
    if (lane == 31) s_w[warp] = inc;
    __syncthreads();
    unsigned long long off = 0, tot = 0;
    for (int w2 = 0; w2 < kBkThreads / 32; w2++) {
        const unsigned long long x = s_w[w2];
        if (w2 < warp) off += x;
        tot += x;
    }
    *total = tot;
    return off + inc - v;
}

// flag[0] of the instance's scratch region: 1 when fullsort_alpha_kernel has to do the row, else 0.
template <typename T>
__global__ void __launch_bounds__(kBkThreads)
bucket_alpha_kernel(const T* __restrict__ q, const T* __restrict__ p, int V, int n, double temp_t, double temp_d,
                    const char* __restrict__ ws, char* __restrict__ scratch, size_t scratch_stride,
                    char* __restrict__ params, int pstride, int force_sort, float* __restrict__ alpha_out,
                    int out_stride, int out_off, int* __restrict__ status_out)
{
    extern __shared__ __align__(16) unsigned char bk_smem[];
    GR_CHECK_FLAG_DECL;
    GR_CHECK_FLAG_INIT;
    unsigned long long* const bt_raw = reinterpret_cast<unsigned long long*>(bk_smem);
    int* const cnt_raw = reinterpret_cast<int*>(bt_raw + 2 * kBkBuckets);
    double* const ckey_raw = reinterpret_cast<double*>(cnt_raw + 2 * kBkBuckets);
    int* const cid_raw = reinterpret_cast<int*>(ckey_raw + kBkMaxCand);
    GR_PTR(unsigned long long) bt = GR_MKPTR(unsigned long long, bt_raw, kBkBuckets, GR_CHECK_FLAG);   // target mass, then exclusive prefix
    GR_PTR(unsigned long long) bd = GR_MKPTR(unsigned long long, bt_raw + kBkBuckets, kBkBuckets, GR_CHECK_FLAG);   // draft mass, ditto
    GR_PTR(int) cnt = GR_MKPTR(int, cnt_raw, kBkBuckets, GR_CHECK_FLAG);            // elements per bucket / fill cursor
    GR_PTR(int) seg = GR_MKPTR(int, cnt_raw + kBkBuckets, kBkBuckets, GR_CHECK_FLAG);   // start of a candidate's segment, -1
    GR_PTR(double) ckey = GR_MKPTR(double, ckey_raw, kBkMaxCand, GR_CHECK_FLAG);    // candidate elements: key,
    GR_PTR(int) cid = GR_MKPTR(int, cid_raw, kBkMaxCand, GR_CHECK_FLAG);            // id,
    GR_PTR(int) sid = GR_MKPTR(int, cid_raw + kBkMaxCand, kBkMaxCand, GR_CHECK_FLAG);   // ids in order
    __shared__ double s_r[4][kBkThreads / 32];
    __shared__ unsigned long long s_w[kBkThreads / 32];
    __shared__ int s_nelem, s_fallback;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long b = blockIdx.x;
    const WsHeader* wh = reinterpret_cast<const WsHeader*>(ws + (size_t)b * ws_stride());
    // (no params block and a status array when called for the optimal acceptance alone)
    Header* hdr = params ? reinterpret_cast<Header*>(params + (size_t)b * pstride) : nullptr;
    int* flag = reinterpret_cast<int*>(scratch + (size_t)b * scratch_stride);
    if (tid == 0 && status_out) status_out[b] = wh->bad != 0 ? GR_BAD_LOGITS : GR_OK;
    if (wh->bad != 0 || force_sort) {
        if (tid == 0) {
            flag[0] = 1;                            // (a bad row returns at once there too)
            if (wh->bad != 0 && status_out) alpha_out[(size_t)b * out_stride + out_off] = nanf("");
        }
        return;
    }
    const T* qrow = q + (size_t)b * V;
    const T* prow = p + (size_t)b * V;
    // (scaled logits as products with the reciprocal temperatures: one rounding away from the quotients the sort
    // uses, which moves alpha* by ~1e-16; every pass here forms them the same way)
    const double rt = 1.0 / temp_t, rd = 1.0 / temp_d;
    // ---- pass 1: maxima of both scaled rows, range of the key d - a
    double mt = -1.0e300, md = -1.0e300, kmax = -1.0e300, kmin = 1.0e300;
#pragma unroll 4
    for (int i = tid; i < V; i += kBkThreads) {
        const double a = (double)load_logit<T>(qrow, i) * rt, d = (double)load_logit<T>(prow, i) * rd;
        mt = fmax(mt, a); md = fmax(md, d); kmax = fmax(kmax, d - a); kmin = fmin(kmin, d - a);
    }
    for (int o = 16; o > 0; o >>= 1) {
        mt = fmax(mt, __shfl_xor_sync(0xffffffffu, mt, o)); md = fmax(md, __shfl_xor_sync(0xffffffffu, md, o));
        kmax = fmax(kmax, __shfl_xor_sync(0xffffffffu, kmax, o)); kmin = fmin(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
    }
    if (lane == 0) { s_r[0][warp] = mt; s_r[1][warp] = md; s_r[2][warp] = kmax; s_r[3][warp] = kmin; }
    for (int c = tid; c < kBkBuckets; c += kBkThreads) { bt[c] = 0ull; bd[c] = 0ull; cnt[c] = 0; seg[c] = -1; }
    if (tid == 0) { s_nelem = 0; s_fallback = 0; }
    __syncthreads();
    for (int w2 = 0; w2 < kBkThreads / 32; w2++) {
        mt = fmax(mt, s_r[0][w2]); md = fmax(md, s_r[1][w2]); kmax = fmax(kmax, s_r[2][w2]); kmin = fmin(kmin, s_r[3][w2]);
    }
    // bucket of a key: floor((kmax - key) * invw), a non-decreasing function of kmax - key in floating point, so
    // every element of a lower bucket comes before every element of a higher one in the ratio order
    const double span = kmax - kmin;
    const double invw = span > 0.0 ? (double)kBkBuckets / (span * (1.0 + 1e-9)) : 0.0;
    // ---- pass 2: bucket masses (integers: the sums do not depend on the order of the atomics)
#pragma unroll 4
    for (int i = tid; i < V; i += kBkThreads) {
        const double a = (double)load_logit<T>(qrow, i) * rt, d = (double)load_logit<T>(prow, i) * rd;
        const int c = min(kBkBuckets - 1, (int)((kmax - (d - a)) * invw));
        atomicAdd(&bt[c], mass_fixed(a, mt));
        atomicAdd(&bd[c], mass_fixed(d, md));
        atomicAdd(&cnt[c], 1);
    }
    __syncthreads();
    // ---- prefixes over the buckets, psi at every boundary, lower bound inside every bucket
    unsigned long long mT[kBkPer], mD[kBkPer], sT = 0, sD = 0;
#pragma unroll
    for (int u = 0; u < kBkPer; u++) { mT[u] = bt[tid * kBkPer + u]; mD[u] = bd[tid * kBkPer + u]; sT += mT[u]; sD += mD[u]; }
    unsigned long long totT, totD;
    unsigned long long pT = block_exscan_u64(sT, s_w, &totT);
    unsigned long long pD = block_exscan_u64(sD, s_w, &totD);
    const double iT = 1.0 / (double)totT, iD = 1.0 / (double)totD;
    // tgt_i / drf_i = exp(-key_i) * rscale
    const double rscale = exp(md - mt) * ((double)totD / (double)totT);
    double lb[kBkPer], best = 0.0;                          // psi of the empty prefix
#pragma unroll
    for (int u = 0; u < kBkPer; u++) {
        const int c = tid * kBkPer + u;
        bt[c] = pT; bd[c] = pD;
        const double T0 = (double)pT * iT, D0 = (double)pD * iD;
        pT += mT[u]; pD += mD[u];
        const double T1 = (double)pT * iT, D1 = (double)pD * iD;
        const double dn = pow(D1, (double)n);
        if (cnt[c] > 0) best = fmin(best, T1 - dn);
        // Inside the bucket every ratio tgt / drf is at least rho (its keys are at most kmax - c w), so a prefix that
        // ends inside it has  psi >= T0 + rho (D - D0) - D^n,  concave in D: its minimum over [D0, D1] is at an end.
        // At D0 that is the previous boundary's psi; at D1 it is the bound below.  The slack covers the rounding of
        // the masses to integers (one unit each).
        const double khi = kmax - (invw > 0.0 ? (double)c / invw * (1.0 - 1e-12) : 0.0);
        const double rho = exp(-khi) * rscale * (1.0 - 1e-9);
        lb[u] = T0 + rho * (D1 - D0) - dn - ((double)(cnt[c] + 1) * iT + 1e-14);
    }
    for (int o = 16; o > 0; o >>= 1) best = fmin(best, __shfl_xor_sync(0xffffffffu, best, o));
    __syncthreads();
    if (lane == 0) s_r[0][warp] = best;
    __syncthreads();
    for (int w2 = 0; w2 < kBkThreads / 32; w2++) best = fmin(best, s_r[0][w2]);
    // ---- candidate buckets: those whose interior could hold a smaller psi
#pragma unroll
    for (int u = 0; u < kBkPer; u++) {
        const int c = tid * kBkPer + u, L = cnt[c];
        if (L >= 2 && lb[u] < best) {
            if (L > kBkMaxPerBucket) s_fallback = 1;
            else {
                const int off = atomicAdd(&s_nelem, L);
                if (off + L > kBkMaxCand) s_fallback = 1;
                else { seg[c] = off; cnt[c] = 0; }
            }
        }
    }
    __syncthreads();
    if (s_fallback) {
        if (tid == 0) flag[0] = 1;
        return;
    }
    // ---- pass 3: the candidates' elements, each bucket into its own segment
    if (s_nelem > 0) {
#pragma unroll 4
        for (int i = tid; i < V; i += kBkThreads) {
            const double a = (double)load_logit<T>(qrow, i) * rt, d = (double)load_logit<T>(prow, i) * rd;
            const int c = min(kBkBuckets - 1, (int)((kmax - (d - a)) * invw));
            if (seg[c] >= 0) {
                const int pos = seg[c] + atomicAdd(&cnt[c], 1);
                ckey[pos] = d - a; cid[pos] = i;
            }
        }
    }
    __syncthreads();
    // ---- one warp per candidate bucket: order by (key descending, id ascending) by counting, then walk the prefixes
    if (s_nelem > 0) {
        for (int c = warp; c < kBkBuckets; c += kBkThreads / 32) {
            const int off = seg[c];
            if (off < 0) continue;
            const int L = cnt[c];
            for (int e = lane; e < L; e += 32) {
                const double ke = ckey[off + e];
                const int ie = cid[off + e];
                int rank = 0;
                for (int j = 0; j < L; j++) {
                    const double kj = ckey[off + j];
                    const int ij = cid[off + j];
                    rank += (kj > ke || (kj == ke && ij < ie)) ? 1 : 0;
                }
                sid[off + rank] = ie;
            }
            __syncwarp();
            unsigned long long cT = bt[c], cD = bd[c];
            for (int base = 0; base < L; base += 32) {
                unsigned long long tf = 0, df = 0;
                if (base + lane < L) {
                    const int id = sid[off + base + lane];
                    tf = mass_fixed((double)load_logit<T>(qrow, id) * rt, mt);
                    df = mass_fixed((double)load_logit<T>(prow, id) * rd, md);
                }
                for (int o = 1; o < 32; o <<= 1) {
                    const unsigned long long t2 = __shfl_up_sync(0xffffffffu, tf, o), d2 = __shfl_up_sync(0xffffffffu, df, o);
                    if (lane >= o) { tf += t2; df += d2; }
                }
                if (base + lane < L)
                    best = fmin(best, (double)(cT + tf) * iT - pow((double)(cD + df) * iD, (double)n));
                cT += __shfl_sync(0xffffffffu, tf, 31); cD += __shfl_sync(0xffffffffu, df, 31);
            }
        }
        for (int o = 16; o > 0; o >>= 1) best = fmin(best, __shfl_xor_sync(0xffffffffu, best, o));
        __syncthreads();
        if (lane == 0) s_r[0][warp] = best;
        __syncthreads();
        for (int w2 = 0; w2 < kBkThreads / 32; w2++) best = fmin(best, s_r[0][w2]);
    }
    __syncthreads();
    if (tid == 0) {
        flag[0] = 0;
        if (hdr) { hdr->alpha_star = 1.0 + best; hdr->resid_total = -best; }
        alpha_out[(size_t)b * out_stride + out_off] = (float)(1.0 + best);
        if (GR_CHECK_VALUE) {                       // (bounds-checked build: an access was out of range)
            if (hdr) hdr->status = GR_CHECK_FAILED;
            if (status_out) status_out[b] = GR_CHECK_FAILED;
            alpha_out[(size_t)b * out_stride + out_off] = nanf("");
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(kFsThreads)
fullsort_alpha_kernel(const T* __restrict__ q, const T* __restrict__ p, int V, int n, double temp_t, double temp_d,
                      const char* __restrict__ ws, char* __restrict__ scratch, char* __restrict__ params, int pstride,
                      float* __restrict__ alpha_out, int out_stride, int out_off)
{
    __shared__ double s_a[kFsThreads / 32], s_b[kFsThreads / 32];
    __shared__ double s_carry[2];
    __shared__ double s_min[kFsThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long b = blockIdx.x;
    const WsHeader* wh = reinterpret_cast<const WsHeader*>(ws + (size_t)b * ws_stride());
    Header* hdr = params ? reinterpret_cast<Header*>(params + (size_t)b * pstride) : nullptr;
    if (wh->bad != 0) return;                       // header / status already say GR_BAD_LOGITS
    const T* qrow = q + (size_t)b * V;
    const T* prow = p + (size_t)b * V;
    const int VP = next_pow2(V);
    unsigned long long* key = reinterpret_cast<unsigned long long*>(scratch + (size_t)b * VP * 12);
    // the first word of the region says whether bucket_alpha_kernel left this row to the sort
    const int todo = reinterpret_cast<const int*>(key)[0];
    __syncthreads();
    if (todo == 0) return;
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
        if (hdr) { hdr->alpha_star = 1.0 + best; hdr->resid_total = -best; }
        alpha_out[(size_t)b * out_stride + out_off] = (float)(1.0 + best);
    }
}

void launch_fullsort(const void* q, const void* p, int dtype, int V, int n, double temp_t, double temp_d, int batch,
                     const char* ws, char* scratch, char* params, int pstride, int force_sort, float* alpha_out,
                     int out_stride, int out_off, int* status_out, cudaStream_t st)
{
    // function attributes belong to the device: set once per device (a failure shows up as a launch error)
    static bool configured[kMaxDevices] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) dev = -1;
    if (dev < 0 || !configured[dev]) {
        const bool ok = cudaFuncSetAttribute(fullsort_alpha_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kFsSmemBytes) == cudaSuccess &&
                        cudaFuncSetAttribute(fullsort_alpha_kernel<__nv_bfloat16>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, kFsSmemBytes) == cudaSuccess &&
                        cudaFuncSetAttribute(bucket_alpha_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kBkSmemBytes) == cudaSuccess &&
                        cudaFuncSetAttribute(bucket_alpha_kernel<__nv_bfloat16>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, kBkSmemBytes) == cudaSuccess;
        if (dev >= 0 && ok) configured[dev] = true;
    }
    const size_t sstride = (size_t)next_pow2(V) * 12;
    if (dtype == GR_F32)
        bucket_alpha_kernel<float><<<batch, kBkThreads, kBkSmemBytes, st>>>((const float*)q, (const float*)p, V, n, temp_t,
                                                                            temp_d, ws, scratch, sstride, params, pstride,
                                                                            force_sort, alpha_out, out_stride, out_off,
                                                                            status_out);
    else
        bucket_alpha_kernel<__nv_bfloat16><<<batch, kBkThreads, kBkSmemBytes, st>>>((const __nv_bfloat16*)q,
                                                                                    (const __nv_bfloat16*)p, V, n, temp_t,
                                                                                    temp_d, ws, scratch, sstride, params,
                                                                                    pstride, force_sort, alpha_out, out_stride,
                                                                                    out_off, status_out);
    if (dtype == GR_F32)
        fullsort_alpha_kernel<float><<<batch, kFsThreads, kFsSmemBytes, st>>>((const float*)q, (const float*)p, V, n, temp_t,
                                                                   temp_d, ws, scratch, params, pstride, alpha_out,
                                                                   out_stride, out_off);
    else
        fullsort_alpha_kernel<__nv_bfloat16><<<batch, kFsThreads, kFsSmemBytes, st>>>((const __nv_bfloat16*)q,
                                                                           (const __nv_bfloat16*)p, V, n, temp_t,
                                                                           temp_d, ws, scratch, params, pstride,
                                                                           alpha_out, out_stride, out_off);
}

}  // namespace gr
