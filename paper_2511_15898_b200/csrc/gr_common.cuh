// Shared device-side definitions of the global-resolution library: the layout of
// the params block and of the workspace, and small helpers.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "gr.h"

namespace gr {

// ---- Bounds-checked build.  Compiled with -DGR_CHECK (paper_2511_15898_b200.build.build_library(check=True), a
// separate library file) every pointer into shared memory, into the workspace records and into the params block
// carries its extent: an access outside it is SKIPPED (a read gives 0) and raises a per-CTA flag, which the kernel
// turns into the instance's status GR_CHECK_FAILED.  It stands in for a memory checker on machines where none may
// run; nothing traps or asserts.  Without the macro the same names are plain pointers and cost nothing.
#ifdef GR_CHECK
template <class T> struct CkNonConst { typedef T type; };
template <class T> struct CkNonConst<const T> { typedef T type; };
template <class T>
struct CkPtr {
    T* p; long long n; int* bad;
    mutable typename CkNonConst<T>::type sink;
    __host__ __device__ CkPtr() : p(nullptr), n(0), bad(nullptr), sink() {}
    __host__ __device__ CkPtr(T* p_, long long n_, int* bad_) : p(p_), n(n_), bad(bad_), sink() {}
    template <class U> __host__ __device__ CkPtr(const CkPtr<U>& o) : p(o.p), n(o.n), bad(o.bad), sink() {}
    __device__ T& operator[](long long i) const {
        if (i >= 0 && i < n) return p[i];
        if (bad) *bad = 1;
        sink = typename CkNonConst<T>::type();
        return sink;
    }
    __device__ T& operator*() const { return (*this)[0]; }
    __host__ __device__ CkPtr operator+(long long k) const { return CkPtr(p + k, n - k, bad); }
    __host__ __device__ CkPtr operator-(long long k) const { return CkPtr(p - k, n + k, bad); }
    template <class U> __host__ __device__ CkPtr<U> as() const {
        return CkPtr<U>(reinterpret_cast<U*>(p), n * (long long)sizeof(T) / (long long)sizeof(U), bad);
    }
};
#define GR_PTR(T) ::gr::CkPtr<T>
#define GR_MKPTR(T, ptr, count, flag) ::gr::CkPtr<T>((ptr), (count), (flag))
#define GR_PCAST(T, ptr) ((ptr).template as<T>())
#define GR_CHECK_FLAG_DECL __shared__ int s_check_flag
#define GR_CHECK_FLAG (&s_check_flag)
#define GR_CHECK_FLAG_INIT do { if (threadIdx.x == 0) s_check_flag = 0; __syncthreads(); } while (0)
#define GR_CHECK_VALUE (s_check_flag)
#else
template <class T> using RawPtr = T*;       // (an alias, so that "GR_PTR(double) a, b;" declares two pointers)
#define GR_PTR(T) ::gr::RawPtr<T>
#define GR_MKPTR(T, ptr, count, flag) (ptr)
#define GR_PCAST(T, ptr) (reinterpret_cast<T*>(ptr))
#define GR_CHECK_FLAG_DECL
#define GR_CHECK_FLAG (nullptr)
#define GR_CHECK_FLAG_INIT do { } while (0)
#define GR_CHECK_VALUE (0)
#endif

constexpr int kMaxSupport = GR_MAX_SUPPORT;   // largest support the convex programs are solved on
constexpr int kMaxDrafts = GR_MAX_DRAFTS;     // largest n
constexpr int kChunk = 1024;                  // elements per chunk of the target-row mass table
constexpr uint32_t kMagic = 0x47525031u;      // "GRP1"

// Header of one instance inside the params block (96 bytes).
struct __align__(16) Header {
    uint32_t magic;
    int V, n, k;              // k = support size (0 when the rule was not solved)
    int jstar, nblocks;       // |H*|, number of outer blocks
    int status, nch;          // solve status, number of chunks in the mass table
    double alpha_star;        // 1 + psi(H*)
    double lse_t;             // log sum exp of target logits / temp_target
    double resid_total;       // total residual mass the resample segment is drawn from
    double gnorm;             // L1 gradient norm at the returned weights (all systems summed)
    const void* q_row;        // this instance's target row
    int dtype, head;          // logits element type; elements before the first 16-byte boundary
    float temp_target;
    int iters;                // gradient evaluations spent (low 16 bits); bit 16: the norm of some system is a prediction
    int kcap;                 // capacity of the per-support arrays
    int stride;               // bytes from one instance's header to the next
};
static_assert(sizeof(Header) == 96, "params header layout");
// The evaluation count a system's solver returns carries, in bit 16, whether its last gradient norm was predicted
// from the final Newton step instead of evaluated; per instance the counts add up and the bits are or-ed.
constexpr int kItersMask = 0xffff;
constexpr int kItersPredicted = 1 << 16;
__host__ __device__ inline int add_iters(int total, int it) {
    return (((total & kItersMask) + (it & kItersMask)) & kItersMask) | ((total | it) & ~kItersMask);
}

// Per-instance params block: Header, then
//   int    id[kcap]     token id in ratio order (position 0 = largest drf/tgt)
//   int    blk[kcap]    -1 on H*, else block number counted from the lowest ratio
//   double w[kcap]      exp(alpha_i)
//   double r[kcap]      outer residual (0 on H*)
//   double p[kcap]      flow p_i = tgt_i - r_i
//   float2 chunk[nchcap]  (max, sum exp2) of target logits per 1024-element chunk
__host__ __device__ inline int round16(int x) { return (x + 15) & ~15; }
__host__ __device__ inline int kcap_of(int V, int topk) {
    int k = (topk <= 0 || topk >= V) ? V : topk;
    return k <= kMaxSupport ? ((k + 3) & ~3) : 0;
}
__host__ __device__ inline int nchcap_of(int V) { return (V + kChunk - 1) / kChunk + 1; }
__host__ __device__ inline int params_stride(int V, int topk) {
    return round16((int)sizeof(Header) + kcap_of(V, topk) * 32 + nchcap_of(V) * 8);
}
struct ParamView {
    Header* h; GR_PTR(int) id; GR_PTR(int) blk; GR_PTR(double) w; GR_PTR(double) r; GR_PTR(double) p; GR_PTR(float2) chunk;
};
// (V and `flag` only matter to the bounds-checked build: extent of the chunk table, where to report)
__host__ __device__ inline ParamView view_params(void* base, int kcap, int V = 1 << 21, int* flag = nullptr) {
    ParamView v;
    char* c = (char*)base;
    v.h = (Header*)c; c += sizeof(Header);
    v.w = GR_MKPTR(double, (double*)c, kcap, flag); c += (size_t)kcap * 8;
    v.r = GR_MKPTR(double, (double*)c, kcap, flag); c += (size_t)kcap * 8;
    v.p = GR_MKPTR(double, (double*)c, kcap, flag); c += (size_t)kcap * 8;
    v.id = GR_MKPTR(int, (int*)c, kcap, flag); c += (size_t)kcap * 4;
    v.blk = GR_MKPTR(int, (int*)c, kcap, flag); c += (size_t)kcap * 4;
    v.chunk = GR_MKPTR(float2, (float2*)c, nchcap_of(V), flag);
    (void)V; (void)flag;
    return v;
}

// Workspace of one instance (written by the scan kernel, read by the solve kernel).
struct __align__(16) WsHeader {
    double lse_t;        // log sum exp of target logits / temp_target
    double lse_d;        // same for the whole draft row (only when the support is the whole vocabulary)
    int count;           // entries that follow (the support, k of them)
    int bad;             // 1 when a non-finite logit was met
    int check;           // bounds-checked build: the streaming kernel skipped an out-of-range access on this row
    int pad;
};
// then: int id[kMaxSupport]; float dl[kMaxSupport]; float tl[kMaxSupport];
__host__ __device__ inline int ws_stride() { return (int)sizeof(WsHeader) + kMaxSupport * 12; }

// alignment head of row b: elements before the first 16-byte boundary
__host__ __device__ inline int row_head(const void* base, long long b, int V, int esize) {
    unsigned long long a = (unsigned long long)base + (unsigned long long)b * (unsigned long long)V * esize;
    int mis = (int)(a & 15ull);
    int head = mis ? (16 - mis) / esize : 0;
    return head < V ? head : V;
}
__host__ __device__ inline int num_chunks(int V, int head) {
    int body = V - head;
    int nch = (body + kChunk - 1) / kChunk;
    return nch < 1 ? 1 : nch;
}
// chunk that holds element i
__device__ inline int chunk_of(int i, int head, int nch) {
    if (i < head) return 0;
    int c = (i - head) / kChunk;
    return c < nch ? c : nch - 1;
}
__device__ inline int chunk_begin(int c, int head) { return c == 0 ? 0 : head + c * kChunk; }
__device__ inline int chunk_end(int c, int head, int nch, int V) {
    if (c == nch - 1) return V;
    int e = head + (c + 1) * kChunk;
    return e < V ? e : V;
}

template <typename T> __device__ inline float load_logit(const T* row, int i);
template <> __device__ inline float load_logit<float>(const float* row, int i) { return __ldg(row + i); }
template <> __device__ inline float load_logit<__nv_bfloat16>(const __nv_bfloat16* row, int i) {
    return __bfloat162float(row[i]);
}
__device__ inline float load_logit_dyn(const void* row, int dtype, int i) {
    return dtype == GR_BF16 ? load_logit<__nv_bfloat16>((const __nv_bfloat16*)row, i)
                            : load_logit<float>((const float*)row, i);
}

// order-preserving map float -> uint32 (larger float, larger key)
__device__ inline uint32_t fkey(float f) {
    uint32_t u = __float_as_uint(f + 0.f);       // (-0 + 0 = +0: the two zeros compare equal, so they get one key)
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ inline float fkey_inv(uint32_t k) {
    uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
    return __uint_as_float(u);
}
// composite key: larger logit first, equal logits: smaller id first
__device__ inline unsigned long long ckey(float v, int id) {
    return ((unsigned long long)fkey(v) << 32) | (unsigned long long)(0xffffffffu - (uint32_t)id);
}

constexpr int kMaxDevices = 64;               // per-device caches of the host code (function attributes, streams)

}  // namespace gr
