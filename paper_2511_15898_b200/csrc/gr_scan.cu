// Streaming pass over the two logit rows of every instance (one CTA per instance).
//
// In a single read of the rows it produces
//   - the log-sum-exp of the target row at temp_target and, per 1024-element chunk,
//     the (max, sum exp2) pair the resample draw later uses as a two-level CDF
//     (distributions from logits: App. A, first paragraph);
//   - the draft support: the `ksel` largest draft logits, equal logits resolved in
//     favour of the smaller id (top-k reduction of the problem, App. N), together
//     with the target logits at those ids.
//
// Selection without a second pass: a threshold tau that is provably not above the
// ksel-th largest draft logit is derived from per-thread running maxima (each of the
// ksel largest thread maxima is a distinct element, so the ksel-th largest of them
// bounds the answer from below); elements >= tau are appended to a shared candidate
// list and the exact answer is taken from the list at the end.  If the list ever
// overflows (adversarially ordered rows) an exact multi-pass radix selection over
// the row replaces it.
#include "gr_common.cuh"

namespace gr {

constexpr int kScanThreads = 512;    // two CTAs per SM: one CTA's epilogue overlaps the other's streaming
constexpr int kScanWarps = kScanThreads / 32;
constexpr int kCandCap = 2048;
constexpr int kMaxChunks = 2049;     // V <= 2^21

template <typename T> struct VecTraits;
template <> struct VecTraits<float> {
    static constexpr int N = 4;
    using Vec = float4;
    __device__ static void unpack(const float4& v, float* o) { o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w; }
};
template <> struct VecTraits<__nv_bfloat16> {
    static constexpr int N = 8;
    using Vec = uint4;
    __device__ static void unpack(const uint4& v, float* o) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; i++) {
            o[2 * i] = __uint_as_float(w[i] << 16);
            o[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// online (max, sum exp2((x-max)*sc)) update with n new values
template <int N>
__device__ __forceinline__ void osm_update(float& m, float& s, const float* x, float sc) {
    float vm = x[0];
#pragma unroll
    for (int i = 1; i < N; i++) vm = fmaxf(vm, x[i]);
    float mn = fmaxf(m, vm);
    float acc = s * ex2((m - mn) * sc);
#pragma unroll
    for (int i = 0; i < N; i++) acc += ex2((x[i] - mn) * sc);
    s = acc; m = mn;
}
__device__ __forceinline__ void osm_merge(float& m, float& s, float mo, float so, float sc) {
    float mn = fmaxf(m, mo);
    // an empty partner (mo = -inf, so = 0) must not poison the sum with inf - inf
    float a = (m == mn) ? s : s * ex2((m - mn) * sc);
    float b = (mo == mn) ? so : so * ex2((mo - mn) * sc);
    s = a + b; m = mn;
}
__device__ __forceinline__ void osm_warp_reduce(float& m, float& s, float sc) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float mo = __shfl_xor_sync(0xffffffffu, m, o);
        float so = __shfl_xor_sync(0xffffffffu, s, o);
        osm_merge(m, s, mo, so, sc);
    }
}

struct CandList {
    GR_PTR(float) v; GR_PTR(int) id; int* cnt;
};
// every lane of the warp calls this; `ok` marks lanes holding a real element
__device__ __forceinline__ void push_one(const CandList& cl, float val, int id, bool ok, float tau, int lane) {
    bool ps = ok && (val >= tau);
    unsigned mk = __ballot_sync(0xffffffffu, ps);
    if (mk == 0) return;
    int leader = __ffs(mk) - 1;
    int base = 0;
    if (lane == leader) base = atomicAdd(cl.cnt, __popc(mk));
    base = __shfl_sync(0xffffffffu, base, leader);
    if (ps) {
        int slot = base + __popc(mk & ((1u << lane) - 1u));
        if (slot < kCandCap) { cl.v[slot] = val; cl.id[slot] = id; }
    }
}

// largest tau (to 16 leading key bits) such that at least `need` threads hold a running maximum >= tau
__device__ float refine_tau(float lmax, int need) {
    uint32_t key = fkey(lmax);
    uint32_t res = 0;
    for (int bit = 31; bit >= 16; bit--) {
        uint32_t t = res | (1u << bit);
        int c = __syncthreads_count(key >= t);
        if (c >= need) res = t;
    }
    return fkey_inv(res);
}

// one lane's element
__device__ __forceinline__ void push_lane(const CandList& cl, float val, int id, float tau) {
    if (val >= tau) {
        const int slot = atomicAdd(cl.cnt, 1);
        if (slot < kCandCap) { cl.v[slot] = val; cl.id[slot] = id; }
    }
}

// Exact selection of the ksel largest composite keys of the draft row by eight 8-bit
// radix passes over the row (slow path, taken only when the candidate list overflowed).
template <typename T>
__device__ void exact_select_slow(const T* prow, int V, int ksel, const CandList& cl, GR_PTR(int) hist /*256 ints*/,
                                  unsigned long long* s_prefix, int* s_need) {
    const int tid = threadIdx.x;
    if (tid == 0) { *s_prefix = 0ull; *s_need = ksel; }
    __syncthreads();
    for (int pass = 0; pass < 8; pass++) {
        const int shift = 56 - 8 * pass;
        for (int i = tid; i < 256; i += kScanThreads) hist[i] = 0;
        __syncthreads();
        const unsigned long long prefix = *s_prefix;
        for (int i = tid; i < V; i += kScanThreads) {
            unsigned long long key = ckey(load_logit<T>(prow, i), i);
            bool match = (pass == 0) || ((key >> (shift + 8)) == (prefix >> (shift + 8)));
            if (match) atomicAdd(&hist[(int)((key >> shift) & 255ull)], 1);
        }
        __syncthreads();
        if (tid == 0) {
            int need = *s_need, acc = 0, bin = 255;
            for (; bin > 0; bin--) {
                if (acc + hist[bin] >= need) break;
                acc += hist[bin];
            }
            *s_need = need - acc;
            *s_prefix = prefix | ((unsigned long long)bin << shift);
        }
        __syncthreads();
    }
    const unsigned long long kth = *s_prefix;     // the ksel-th largest composite key (keys are distinct)
    if (tid == 0) *cl.cnt = 0;
    __syncthreads();
    for (int i = tid; i < V; i += kScanThreads) {
        float v = load_logit<T>(prow, i);
        if (ckey(v, i) >= kth) {
            int slot = atomicAdd(cl.cnt, 1);
            if (slot < kCandCap) { cl.v[slot] = v; cl.id[slot] = i; }
        }
    }
    __syncthreads();
}

// kFull: the support is the whole vocabulary and exceeds kMaxSupport; no support is
// selected, the draft row's log-sum-exp is produced instead.
template <typename T, bool kFull>
__global__ void __launch_bounds__(kScanThreads, 2)
scan_kernel(const T* __restrict__ q, const T* __restrict__ p, int V, int ksel, float sc_t, float sc_d,
            double temp_t, double temp_d, char* __restrict__ ws, char* __restrict__ params, int pstride, int kcap)
{
    using VT = VecTraits<T>;
    constexpr int N = VT::N;
    constexpr int S = kChunk / (32 * N);   // vector steps per chunk and warp
    constexpr int U = 4;                   // steps in flight
    constexpr int NB = S / U;
    static_assert(S % U == 0, "chunk must be a whole number of batches");

    __shared__ unsigned long long s_keys_raw[kCandCap];
    __shared__ float2 s_chunk_raw[kMaxChunks];
    __shared__ float s_dm[kScanWarps], s_ds[kScanWarps];
    __shared__ int s_hist_raw[256];
    GR_CHECK_FLAG_DECL;
    GR_CHECK_FLAG_INIT;
    GR_PTR(unsigned long long) s_keys = GR_MKPTR(unsigned long long, s_keys_raw, kCandCap, GR_CHECK_FLAG);
    GR_PTR(float2) s_chunk = GR_MKPTR(float2, s_chunk_raw, kMaxChunks, GR_CHECK_FLAG);
    GR_PTR(int) s_hist = GR_MKPTR(int, s_hist_raw, 256, GR_CHECK_FLAG);
    __shared__ unsigned long long s_prefix;
    __shared__ int s_need, s_cnt, s_bad;
    __shared__ float s_tau;
    __shared__ double s_lse[2];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long b = blockIdx.x;
    const T* qrow = q + (size_t)b * V;
    const T* prow = p + (size_t)b * V;
    const int head = row_head(q, b, V, (int)sizeof(T));
    const int nch = num_chunks(V, head);
    const int vec_end = head + ((V - head) / N) * N;
    const int tail = V - vec_end;

    CandList cl;
    cl.v = GR_MKPTR(float, reinterpret_cast<float*>(s_keys_raw), kCandCap, GR_CHECK_FLAG);
    cl.id = GR_MKPTR(int, reinterpret_cast<int*>(s_keys_raw) + kCandCap, kCandCap, GR_CHECK_FLAG);
    cl.cnt = &s_cnt;
    const bool take_all = !kFull && (V <= kCandCap);       // every element is a candidate
    const bool use_tau = !kFull && !take_all;
    if (tid == 0) { s_cnt = 0; s_bad = 0; s_tau = -INFINITY; }
    __syncthreads();

    float lmax = -INFINITY;            // running maximum of this thread's draft logits
    float dm = -INFINITY, dsum_e = 0.f;   // draft row (kFull only)
    float tsum = 0.f, dsum = 0.f;      // plain sums: any NaN / inf makes them non-finite
    const int rounds = (nch + kScanWarps - 1) / kScanWarps;

    for (int r = 0; r < rounds; r++) {
        const int c = r * kScanWarps + warp;
        const bool cvalid = c < nch;
        float cm = -INFINITY, cs = 0.f;     // this lane's share of chunk c
        // scalar head / tail elements join their chunk here (their candidates are pushed at the end)
        if (cvalid && c == 0 && lane < head) {
            float x = load_logit<T>(qrow, lane), v = load_logit<T>(prow, lane);
            osm_update<1>(cm, cs, &x, sc_t);
            tsum += x; dsum += v; lmax = fmaxf(lmax, v);
            if (kFull) osm_update<1>(dm, dsum_e, &v, sc_d);
        }
        if (cvalid && c == nch - 1 && lane < tail) {
            float x = load_logit<T>(qrow, vec_end + lane), v = load_logit<T>(prow, vec_end + lane);
            osm_update<1>(cm, cs, &x, sc_t);
            tsum += x; dsum += v; lmax = fmaxf(lmax, v);
            if (kFull) osm_update<1>(dm, dsum_e, &v, sc_d);
        }
        // Batches of U vector steps.  A candidate (draft logit >= tau) is appended by its own lane, without any warp
        // vote: about one element in four hundred is one, and the list's order does not matter (the exact selection
        // sorts it).  The CTA's very first batch has no threshold yet: it derives one afterwards and reads its
        // draft vectors once more (from cache) to test them.
#pragma unroll 1
        for (int nb = 0; nb < NB; nb++) {
            typename VT::Vec qv[U], pv[U];
            int idx[U];
            bool ok[U];
#pragma unroll
            for (int u = 0; u < U; u++) {
                idx[u] = head + c * kChunk + ((nb * U + u) * 32 + lane) * N;
                ok[u] = cvalid && (idx[u] + N <= vec_end);
#ifdef GR_CHECK
                if (ok[u] && (idx[u] < 0 || idx[u] + N > V || ((size_t)(qrow + idx[u]) & 15))) { s_check_flag = 1; ok[u] = false; }
#endif
                if (ok[u]) {
                    qv[u] = __ldcs(reinterpret_cast<const typename VT::Vec*>(qrow + idx[u]));
                    pv[u] = __ldcs(reinterpret_cast<const typename VT::Vec*>(prow + idx[u]));
                }
            }
            const bool sample = use_tau && (r == 0) && (nb == 0);
            // (+inf on the first batch: nothing passes the in-loop test)
            const float tau = sample ? INFINITY : (use_tau ? *((volatile float*)&s_tau) : -INFINITY);
#pragma unroll
            for (int u = 0; u < U; u++) {
                if (ok[u]) {
                    float tv[N], dv[N];
                    VT::unpack(qv[u], tv);
                    VT::unpack(pv[u], dv);
                    osm_update<N>(cm, cs, tv, sc_t);
                    if (kFull) osm_update<N>(dm, dsum_e, dv, sc_d);
                    float vm = dv[0];
#pragma unroll
                    for (int i = 0; i < N; i++) { tsum += tv[i]; dsum += dv[i]; vm = fmaxf(vm, dv[i]); }
                    lmax = fmaxf(lmax, vm);
                    if (!kFull && vm >= tau) {
#pragma unroll
                        for (int i = 0; i < N; i++) push_lane(cl, dv[i], idx[u] + i, tau);
                    }
                }
            }
            if (!kFull && sample) {
                float t0 = refine_tau(lmax, ksel);      // contains CTA-wide barriers; every warp gets here
                if (tid == 0) s_tau = fmaxf(s_tau, t0);
                __syncthreads();
                const float tau1 = *((volatile float*)&s_tau);
                for (int u = 0; u < U; u++) {
                    if (ok[u]) {
                        float dv[N];
                        VT::unpack(*reinterpret_cast<const typename VT::Vec*>(prow + idx[u]), dv);
#pragma unroll
                        for (int i = 0; i < N; i++) push_lane(cl, dv[i], idx[u] + i, tau1);
                    }
                }
            }
        }
        // chunk result
        osm_warp_reduce(cm, cs, sc_t);
        if (cvalid && lane == 0) s_chunk[c] = make_float2(cm, cs);
        if (use_tau && r < 4 && r + 1 < rounds) {
            float t1 = refine_tau(lmax, ksel);
            if (tid == 0) s_tau = fmaxf(s_tau, t1);
            __syncthreads();
        }
    }
    // candidates among the scalar head / tail elements
    if (!kFull && warp == 0) {
        float tau = use_tau ? *((volatile float*)&s_tau) : -INFINITY;
        bool okh = lane < head;
        float vh = okh ? load_logit<T>(prow, lane) : -INFINITY;
        push_one(cl, vh, lane, okh, tau, lane);
        bool okt = lane < tail;
        float vt = okt ? load_logit<T>(prow, vec_end + lane) : -INFINITY;
        push_one(cl, vt, vec_end + lane, okt, tau, lane);
    }
    // non-finite inputs
    {
        bool badl = !(fabsf(tsum) <= 3.0e38f) || !(fabsf(dsum) <= 3.0e38f);
        if (__any_sync(0xffffffffu, badl) && lane == 0) atomicOr(&s_bad, 1);
    }
    if (kFull) {
        osm_warp_reduce(dm, dsum_e, sc_d);
        if (lane == 0) { s_dm[warp] = dm; s_ds[warp] = dsum_e; }
    }
    __syncthreads();

    // ---- row totals in fp64 from the chunk table (so that the chunk masses sum to one)
    if (warp == 0) {
        double M = -INFINITY;
        for (int c = lane; c < nch; c += 32) M = fmax(M, (double)s_chunk[c].x);
        for (int o = 16; o > 0; o >>= 1) M = fmax(M, __shfl_xor_sync(0xffffffffu, M, o));
        double acc = 0.0;
        for (int c = lane; c < nch; c += 32)
            acc += (double)s_chunk[c].y * exp(((double)s_chunk[c].x - M) / temp_t);
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) {
            s_lse[0] = M / temp_t + log(acc);
            if (kFull) {
                double Md = -INFINITY;
                for (int w2 = 0; w2 < kScanWarps; w2++) Md = fmax(Md, (double)s_dm[w2]);
                double ad = 0.0;
                for (int w2 = 0; w2 < kScanWarps; w2++)
                    if (s_ds[w2] > 0.f) ad += (double)s_ds[w2] * exp(((double)s_dm[w2] - Md) / temp_d);
                s_lse[1] = Md / temp_d + log(ad);
            } else {
                s_lse[1] = 0.0;
            }
            if (!isfinite(s_lse[0]) || (kFull && !isfinite(s_lse[1]))) s_bad = 1;
        }
    }
    __syncthreads();

    // ---- exact support out of the candidate list
    int nsel = 0;
    if (!kFull) {
        int M = s_cnt;
        nsel = ksel < V ? ksel : V;
        if (M > kCandCap) {
            exact_select_slow<T>(prow, V, nsel, cl, s_hist, &s_prefix, &s_need);
            M = s_cnt;
        }
        if (M > kCandCap) M = kCandCap;
        // composite keys in place of the (value, id) pairs
        constexpr int kPer = kCandCap / kScanThreads;
        float vv[kPer]; int ii[kPer];
#pragma unroll
        for (int u = 0; u < kPer; u++) {
            const int e = tid + u * kScanThreads;
            vv[u] = 0.f; ii[u] = 0;
            if (e < M) { vv[u] = cl.v[e]; ii[u] = cl.id[e]; }
        }
        __syncthreads();
#pragma unroll
        for (int u = 0; u < kPer; u++) {
            const int e = tid + u * kScanThreads;
            if (e < M) s_keys[e] = ckey(vv[u], ii[u]);
        }
        __syncthreads();
        char* wsb = ws + (size_t)b * ws_stride();
        int* w_id_raw = reinterpret_cast<int*>(wsb + sizeof(WsHeader));
        float* w_dl_raw = reinterpret_cast<float*>(w_id_raw + kMaxSupport);
        GR_PTR(int) w_id = GR_MKPTR(int, w_id_raw, kMaxSupport, GR_CHECK_FLAG);
        GR_PTR(float) w_dl = GR_MKPTR(float, w_dl_raw, kMaxSupport, GR_CHECK_FLAG);
        GR_PTR(float) w_tl = GR_MKPTR(float, w_dl_raw + kMaxSupport, kMaxSupport, GR_CHECK_FLAG);
        if (M < nsel) nsel = M;   // cannot happen for finite rows; keeps the writes in range
#pragma unroll
        for (int u = 0; u < kPer; u++) {
            const int e = tid + u * kScanThreads;
            if (e < M) {
                const unsigned long long me = s_keys[e];
                int rank = 0;
                for (int j = 0; j < M; j++) rank += (s_keys[j] > me) ? 1 : 0;
                if (rank < nsel) {
                    w_id[rank] = ii[u];
                    w_dl[rank] = vv[u];
#ifdef GR_CHECK
                    if (ii[u] < 0 || ii[u] >= V) { s_check_flag = 1; ii[u] = 0; }
#endif
                    w_tl[rank] = load_logit<T>(qrow, ii[u]);
                }
            }
        }
    }

    // ---- outputs: workspace header, chunk table and the header fields owned by this kernel
    // (params == nullptr: the caller wants the workspace record only)
    char* pb = params ? params + (size_t)b * pstride : nullptr;
    if (pb) {
        ParamView pv = view_params(pb, kcap, V, GR_CHECK_FLAG);
        for (int c = tid; c < nch; c += kScanThreads) pv.chunk[c] = s_chunk[c];
    }
#ifdef GR_CHECK
    __syncthreads();
#endif
    if (tid == 0) {
        WsHeader* wh = reinterpret_cast<WsHeader*>(ws + (size_t)b * ws_stride());
        wh->lse_t = s_lse[0];
        wh->lse_d = s_lse[1];
        wh->count = nsel;
        wh->bad = s_bad;
        wh->check = GR_CHECK_VALUE;
    }
    if (params == nullptr) return;
    ParamView pv = view_params(pb, kcap, V, GR_CHECK_FLAG);
    if (tid == 0) {
        Header* h = pv.h;
        h->magic = 0;            // completed by the solve kernel
        h->V = V; h->nch = nch; h->head = head;
        h->q_row = qrow;
        h->dtype = sizeof(T) == 2 ? GR_BF16 : GR_F32;
        h->lse_t = s_lse[0];
        h->temp_target = (float)temp_t;
        h->kcap = kcap; h->stride = pstride;
    }
}

void launch_scan(const void* q, const void* p, int dtype, int V, int ksel, bool full_large, double temp_t,
                 double temp_d, int batch, char* ws, char* params, int pstride, int kcap, cudaStream_t st)
{
    const double log2e = 1.4426950408889634;
    float sc_t = (float)(log2e / temp_t), sc_d = (float)(log2e / temp_d);
    dim3 grid(batch), block(kScanThreads);
    if (dtype == GR_F32) {
        if (full_large)
            scan_kernel<float, true><<<grid, block, 0, st>>>((const float*)q, (const float*)p, V, ksel, sc_t, sc_d,
                                                               temp_t, temp_d, ws, params, pstride, kcap);
        else
            scan_kernel<float, false><<<grid, block, 0, st>>>((const float*)q, (const float*)p, V, ksel, sc_t, sc_d,
                                                                temp_t, temp_d, ws, params, pstride, kcap);
    } else {
        if (full_large)
            scan_kernel<__nv_bfloat16, true><<<grid, block, 0, st>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)p,
                                                                       V, ksel, sc_t, sc_d, temp_t, temp_d, ws, params,
                                                                       pstride, kcap);
        else
            scan_kernel<__nv_bfloat16, false><<<grid, block, 0, st>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)p,
                                                                        V, ksel, sc_t, sc_d, temp_t, temp_d, ws, params,
                                                                        pstride, kcap);
    }
}

}  // namespace gr
