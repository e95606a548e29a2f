/*
 * gr.h -- C interface of the B200 (sm_100a) global-resolution library.
 *
 * For a batch of decode positions the library turns target logits, draft logits
 * and the number n of i.i.d. drafts into the optimal-transport verification rule
 * of "Global Resolution" (optimal multi-draft speculative sampling) and then
 * draws the emitted token for the n drafted tokens.
 *
 * Letters.  The paper writes p for the target distribution and q for the draft
 * distribution; this interface uses the opposite letters, as serving stacks do:
 *   q_logits = TARGET model logits,  p_logits = DRAFT model logits.
 * In the comments below "tgt" is the target distribution after temperature and
 * "drf" the single-token draft distribution after temperature, top-k truncation
 * and renormalisation (App. A, first paragraph; App. N).
 *
 * Conventions shared by every call
 *   - every pointer named below is a DEVICE pointer owned by the caller unless
 *     it is marked "host"; the library never allocates or frees device memory;
 *   - calls only enqueue work on `stream` (a cudaStream_t passed as void*) and
 *     return without synchronising;
 *   - the int return value is 0 (GR_OK) when the work was enqueued, or a negative
 *     GR_E_* code when the arguments were rejected on the host (nothing enqueued);
 *   - data-dependent outcomes are reported per instance in the status arrays.
 */
#ifndef GR_H_
#define GR_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

/* element type of the logits */
#define GR_F32  0
#define GR_BF16 1

/* per-instance status values (status arrays, device memory) */
#define GR_OK                    0
#define GR_NOT_CONVERGED         1  /* iteration cap reached; the rule is usable, its gradient norm is in params */
#define GR_SUPPORT_TOO_LARGE     2  /* support larger than GR_MAX_SUPPORT: no rule was solved; gr_verify falls
                                       back to sampling the target distribution (still lossless), the paper's
                                       "early termination" convention (Sec. 6.2 last paragraph, App. K)   */
#define GR_BAD_LOGITS            3  /* a NaN or infinite logit in the row                                 */
#define GR_DRAFT_OUT_OF_SUPPORT  4  /* a drafted token does not belong to the draft support               */
#define GR_STALE_PARAMS          5  /* params block was not written by gr_solve for this shape            */
#define GR_PARTIAL_RULE          6  /* params written by gr_solve_verify: only the system its drafted tuple
                                       selects was solved; gr_verify refuses such a block (token -1)       */
#define GR_CHECK_FAILED          7  /* bounds-checked build of the library only: a kernel skipped an access
                                       outside an array's extent while it worked on this instance          */

/* host-side argument errors (return values) */
#define GR_E_INVALID   (-1)  /* a size, temperature or option is out of range */
#define GR_E_NULL      (-2)  /* a required pointer is NULL                    */
#define GR_E_ALIGN     (-3)  /* a logits base pointer is not 16-byte aligned  */
#define GR_E_LAUNCH    (-4)  /* the CUDA runtime refused a launch             */
#define GR_E_TOO_LARGE (-5)  /* beyond a stated capacity                      */

/* capacities */
#define GR_MAX_SUPPORT 128   /* largest draft support for which the convex programs are solved */
#define GR_MAX_DRAFTS  32    /* largest n                                                     */

/*
 * Solver options (host struct, read during the call).  NULL selects the defaults.
 *   tol        stop when the L1 norm of the gradient of the convex function
 *              (Theta for the inner system, Phi restricted to a block for the outer
 *              system; Sec. 6.2) is <= tol.                      default 3e-7
 *              (The default sits just below the ~4.5e-7 that fp32 summation over a
 *              128k-token row leaves in the target's log-sum-exp, i.e. below the
 *              accuracy to which the target distribution itself is known; the emitted
 *              token's law then differs from that target by at most tol in L1.  Smaller
 *              values are honoured down to the quadrature floor of a few 1e-9 at the
 *              default quad_step.)
 *              The kernels also stop after a Newton step taken from a point evaluated
 *              on the full quadrature grid when the residual that step leaves is
 *              predicted below tol, in one of two ways: the step's second-order size
 *              s2 = sum_i g_i (delta alpha_i)^2 ten times below tol (the residual after
 *              such a step stayed within 8.5 s2 + 3e-9 on every shape measured; the
 *              reported gradient norm is then 3 s2), or, after a step that contracted the
 *              residual by rho < 0.1, 3 rho r_k below tol (reported: rho r_k; the faster
 *              kernels only).  Neither is
 *              used when the factorisation of the Newton system left less than 2 % of a
 *              diagonal entry as its pivot (a system too close to singular in fp32).
 *   max_iters  cap on gradient evaluations per system.            default 40
 *   quad_step  step of the trapezoid rule in the log-time variable used to
 *              evaluate the gradient integral; smaller is more accurate and
 *              slower (error roughly exp(-pi^2/quad_step)).        default 0.4
 *   scan_done_event  optional cudaEvent_t (as void*) recorded on `stream` between
 *              the streaming kernel and the solve kernel, so that a caller can
 *              time the two separately; NULL records nothing.      default NULL
 *   force_robust  non-zero sends every shape to the general (slower) solve kernel;
 *              by default supports of at most 128 tokens with n <= 16 take a faster
 *              kernel that computes the same rule.  For an untruncated draft on a
 *              vocabulary beyond GR_MAX_SUPPORT (optimal acceptance only) it selects the
 *              whole-row sort instead of the bucketed search.         default 0
 *   tau        error threshold of Algorithm 1 (Sec. 6.2 "tunable errors", Sec. 6.3).  0 solves the
 *              convex programs on the whole support (the default: both tunable errors are 0 and `tol`
 *              is the stopping rule).  tau in (0, 1] selects the truncated variant: the inner system
 *              is solved on the fewest tokens T of H* with gamma_T = drf(H*)^n - drf(T)^n <= tau, every
 *              outer block on the fewest outer tokens T with epsilon_T = 1 - (drf(H*) + drf(T))^n <= tau
 *              (largest drf first), each to gradient norm 5 tau (`tol` is then not used); tokens outside
 *              the sets keep weight 0 (a tuple served only by such tokens of an outer block is shared
 *              equally among them).  The emitted token then follows the target within 15 tau in L1 and
 *              the acceptance is within 10 tau of alpha* (Lemma "Approximation Guarantee").     default 0
 */
typedef struct gr_options {
    double tol;
    int    max_iters;
    double quad_step;
    void*  scan_done_event;
    int    force_robust;
    double tau;
} gr_options;

/*
 * Bytes of the opaque per-batch `params` block that gr_solve writes and
 * gr_verify reads, and of the scratch `workspace` gr_solve needs while it runs.
 * Both depend only on the shape.  Return 0 when the shape is invalid.
 */
size_t gr_params_bytes(int V, int n, int topk, int batch);
size_t gr_workspace_bytes(int V, int n, int topk, int batch);

/*
 * gr_solve -- steps 1-3 of Algorithm 1 for every instance of the batch.
 *
 * Per instance (one decode position):
 *   tgt = softmax(q_logits / temp_target) over the whole vocabulary;
 *   support = the `topk` largest draft logits (equal logits: the smaller id is
 *   kept), drf = softmax(p_logits / temp_draft) over the support (App. N);
 *   H* and the optimal acceptance alpha* = 1 + min_H psi(H) by ordering the
 *   support by decreasing drf/tgt and scanning prefixes (Eq. "subset-select",
 *   Sec. 5.1; ties: smaller id first, shortest minimising prefix);
 *   outer residuals by cumulative minima of psi along the increasing-ratio
 *   chain (Sec. 6.1, Thm "polymatroid", Lemma "q-convex");
 *   softmax parameters exp(alpha_i) of the inner system on H* (Thm "Inner
 *   Convex Solver") and of every block of the outer system (Thm "Outer Convex
 *   Solver" restricted to the tokens between two consecutive tight prefixes),
 *   with the full truncation set T (tunable errors epsilon_T = gamma_T = 0).
 *
 * Arguments
 *   q_logits, p_logits  [batch, V] row-major, dtype GR_F32 (float) or GR_BF16;
 *                       base pointers 16-byte aligned; read only.
 *   V >= 1, 1 <= n <= GR_MAX_DRAFTS, batch >= 0.
 *   topk                1..V-1 truncates the draft; 0 or >= V keeps every id.
 *   temp_target, temp_draft   > 0.
 *   opt                 host pointer or NULL.
 *   params              out, gr_params_bytes() bytes, 16-byte aligned.  It records
 *                       the address of q_logits: gr_verify re-reads at most one
 *                       1024-element chunk of a target row on the resample branch,
 *                       so q_logits must stay unchanged until gr_verify has run.
 *   workspace           scratch, gr_workspace_bytes() bytes, 16-byte aligned;
 *                       contents are meaningless after the call completes.
 *   alpha_star          out [batch] float, optimal acceptance probability (also produced, by a sort of
 *                       the whole row, when the support exceeds GR_MAX_SUPPORT and no rule is solved).
 *   status              out [batch] int, GR_OK / GR_NOT_CONVERGED /
 *                       GR_SUPPORT_TOO_LARGE / GR_BAD_LOGITS.
 */
int gr_solve(const void* q_logits, const void* p_logits, int dtype, int V, int n, int topk,
             float temp_target, float temp_draft, int batch, const gr_options* opt,
             void* params, void* workspace, float* alpha_star, int* status, void* stream);

/*
 * gr_solve_static -- gr_solve without the `workspace` argument, for callers that cannot
 * allocate device memory.  (The paper has no counterpart: this is an interface variant.)
 *
 * Who needs it: a serving loop that has handed all free device memory to its own pool
 * (KV cache, activation arena) and therefore must not call cudaMalloc at steady state --
 * the call may fail there and it synchronises the whole device -- or a host that is not
 * allowed to allocate at all once it is running (latency-bounded control loops).  Such a
 * caller still owns `params` and the outputs, but has nowhere to take scratch from.
 *
 * The scratch is a fixed array inside the library's device image, GR_STATIC_MAX_BATCH
 * instances large (about 0.4 MB, held by every GPU that loads the library until exit).
 *   - batch > GR_STATIC_MAX_BATCH returns GR_E_TOO_LARGE and launches nothing; split the batch.
 *     So does an untruncated draft on a vocabulary larger than GR_MAX_SUPPORT (its alpha* needs a
 *     per-row sort buffer the built-in scratch does not have).
 *   - The first call on each device looks the array's device address up (that device must
 *     be current, as for any launch); make that first call before any stream capture.
 *   - The call itself allocates and frees nothing.
 *   - All calls share the one array and it keeps the previous call's contents.  Nothing in it
 *     needs clearing (each call rewrites all it reads), but two calls whose kernels overlap on
 *     the GPU -- different streams, or different host threads -- race on it: serialise them.
 * Every other argument, the outputs and the statuses are exactly those of gr_solve, and
 * gr_verify / gr_read_rule take the resulting `params` unchanged.
 */
#define GR_STATIC_MAX_BATCH 256
int gr_solve_static(const void* q_logits, const void* p_logits, int dtype, int V, int n, int topk,
                    float temp_target, float temp_draft, int batch, const gr_options* opt,
                    void* params, float* alpha_star, int* status, void* stream);

/*
 * gr_verify -- step 4 of Algorithm 1 (the slice pi(.|omega), Eqs. "cases" and
 * "approx-c", normalised) and the draw of App. A steps 3-4.
 *
 * Per instance, U = distinct drafted tokens in order of first occurrence.
 * If U lies in H*: pi(i) = w_i / (1 + sum_U w) and the rest, 1 / (1 + sum_U w), goes
 * to the resample distribution (residuals / (1 - alpha*)); otherwise only the
 * tokens of the lowest-ratio block met by U share the mass, pi(i) = w_i / sum w.
 * The emitted token is the first segment (U's tokens in order, then the resample
 * segment) whose cumulative probability exceeds u0; inside the resample segment
 * it is the first id (ascending) whose cumulative residual exceeds u1 times the
 * total residual.
 *
 *   params        written by gr_solve for the same batch; read only.
 *   draft_tokens  [batch, n] int32 (n as given to gr_solve).
 *   uniforms      [batch, 2] float in [0,1): (u0, u1).
 *   out_token     out [batch] int32 emitted id, -1 on a per-instance error.
 *   out_accepted  out [batch] 1 iff the emitted token is one of the drafts.
 *   status        out [batch] GR_OK / GR_DRAFT_OUT_OF_SUPPORT / GR_STALE_PARAMS /
 *                 GR_BAD_LOGITS, or the solve status when it was not GR_OK.
 */
int gr_verify(const void* params, const int* draft_tokens, const float* uniforms, int batch,
              int* out_token, unsigned char* out_accepted, int* status, void* stream);

/*
 * gr_solve_verify -- gr_solve and gr_verify in one call for drafts known beforehand:
 * the solve kernel of every instance looks at its drafted tuple, solves only the
 * system that tuple selects (Eq. "cases": the inner system when every drafted token
 * lies in H*, else the lowest-ratio outer block the tuple meets; Algorithm 1 does the
 * same) and finishes with the draw itself, so no separate verification launch and no
 * second read of the rule.  Arguments as for gr_solve and gr_verify; `status` holds
 * what gr_verify would report.  alpha_star is written as by gr_solve.  The params block
 * is still written (for gr_read_rule); instances where a system was skipped carry
 * GR_PARTIAL_RULE in it and must not be given to gr_verify with other drafts.
 * Same return values as gr_solve.
 */
int gr_solve_verify(const void* q_logits, const void* p_logits, int dtype, int V, int n, int topk,
                    float temp_target, float temp_draft, int batch, const gr_options* opt,
                    const int* draft_tokens, const float* uniforms, void* params, void* workspace,
                    float* alpha_star, int* out_token, unsigned char* out_accepted, int* status,
                    void* stream);

/*
 * gr_alpha_star -- the optimal acceptance alpha* = 1 + min_H psi(H) alone (Eq. "subset-select"), for up to
 * GR_MAX_ALPHA_N draft counts at once: one pass over the logits (the same streaming kernel as gr_solve) and a
 * prefix scan along the ratio order, which all the draft counts share.  No rule is solved and no params block
 * is written; this is what an acceptance-versus-(n, k) sweep needs.
 *   n_list      HOST array of n_count draft counts, each in 1..GR_MAX_DRAFTS.
 *   workspace   scratch of gr_workspace_bytes(V, 1, topk, batch) bytes, 16-byte aligned.
 *   alpha_star  out [batch, n_count] float, row-major; NaN where status is not GR_OK.
 *   status      out [batch]: GR_OK or GR_BAD_LOGITS.
 * Supports: top-k up to GR_MAX_SUPPORT, or the whole vocabulary of any size (beyond GR_MAX_SUPPORT tokens
 * the minimum of psi is searched per draft count without sorting the row, as in gr_solve); a top-k beyond
 * GR_MAX_SUPPORT on a larger vocabulary returns GR_E_TOO_LARGE.
 * Other return values as gr_solve.
 */
#define GR_MAX_ALPHA_N 8
int gr_alpha_star(const void* q_logits, const void* p_logits, int dtype, int V, const int* n_list, int n_count,
                  int topk, float temp_target, float temp_draft, int batch, void* workspace,
                  float* alpha_star, int* status, void* stream);

/*
 * gr_read_rule -- copies the rule of every instance out of `params` into plain
 * arrays (for inspection and tests); all outputs are optional (NULL skips).
 * Per-support arrays have `kcap` entries per instance and are filled in ratio
 * order (position 0 = largest drf/tgt); unused entries are set to -1 / 0.
 *   ids    [batch,kcap] int   token id          w   [batch,kcap] double exp(alpha_i)
 *   block  [batch,kcap] int   -1 on H*, else block number counted from the lowest ratio
 *   resid  [batch,kcap] double outer residual r_i (0 on H*)
 *   flow   [batch,kcap] double p_i = tgt_i - r_i
 *   header [batch,8] double: k, jstar, nblocks, alpha_star, gnorm, iterations, lse of the target row, status
 *          (iterations = gradient evaluations spent, plus 65536 when the gradient norm of at least one of the
 *          instance's convex programs is a prediction from its last Newton step rather than an evaluation)
 */
int gr_read_rule(const void* params, int batch, int kcap, int* ids, int* block, double* w,
                 double* resid, double* flow, double* header, void* stream);

/*
 * gr_read_slice -- the slice pi(.|omega) of every instance for its drafted tuple (Eq. "cases" and Eq. "approx-c",
 * "normalized" as in Algorithm 1), computed by the same device code gr_verify draws from, for inspection and tests:
 * what gr_verify compares u0 with, without the draw.
 *   params        written by gr_solve (not by gr_solve_verify) for the same batch; read only.
 *   draft_tokens  [batch, n] int32, n as given to gr_solve.
 *   U    out [batch, n] int32: U[b, s] = drafted token s of instance b, or -1 when it repeats an earlier one.
 *   pi   out [batch, n] double: probability that token is emitted (0 for repeats, and for tokens outside the
 *        block that serves the tuple); the accepted segments of the draw are these, in this order.
 *   rho  out [batch] double: mass of the resample segment (1 / (1 + sum of the weights) when every drafted token
 *        lies in H*, else 0).
 *   status out [batch]: GR_OK / GR_NOT_CONVERGED (slice given), or GR_DRAFT_OUT_OF_SUPPORT /
 *        GR_SUPPORT_TOO_LARGE / GR_BAD_LOGITS / GR_PARTIAL_RULE / GR_STALE_PARAMS (no slice: U = -1, pi = 0).
 */
int gr_read_slice(const void* params, const int* draft_tokens, int batch, int n, int* U, double* pi,
                  double* rho, int* status, void* stream);

/* Text for a GR_* / GR_E_* code (host pointer to a static string). */
const char* gr_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* GR_H_ */
