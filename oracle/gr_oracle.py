"""ctypes front end of the C oracle (test infrastructure only).

Nothing here computes: every function marshals numpy arrays into the C routines
of gr_oracle.c and returns their outputs.
"""
from __future__ import annotations

import ctypes as C
import dataclasses
from typing import Optional

import numpy as np

from .build import build_oracle

_lib = None

GRO_OK = 0
GRO_NOT_CONVERGED = 1
GRO_BAD_ARG = -1
GRO_DRAFT_OUT_OF_SUPPORT = -2

ROUTE_G1 = 1   # grouped terms, inclusion-exclusion (exponential; small supports)
ROUTE_G2 = 2   # one-dimensional integral
METHOD_IPF = 1     # proportional fitting sweeps only
METHOD_NEWTON = 2  # damped Newton steered by a finite-difference Jacobian


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build_oracle())
    return _lib


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t))


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def distributions(tl, dl, topk, Tt, Td):
    tl, dl = _f64(tl), _f64(dl)
    V = tl.shape[0]
    tgt = np.empty(V)
    drf = np.empty(V)
    ids = np.empty(V, dtype=np.int32)
    lse = C.c_double(0)
    k = lib().gro_distributions(_p(tl, C.c_double), _p(dl, C.c_double), V, int(topk), C.c_double(Tt),
                                C.c_double(Td), _p(tgt, C.c_double), _p(drf, C.c_double), _p(ids, C.c_int),
                                C.byref(lse))
    if k < 0:
        raise ValueError("bad argument")
    return tgt, drf, ids[:k].copy(), lse.value


def alpha_star_only(tl, dl, n, topk, Tt=1.0, Td=1.0):
    """Optimal acceptance and |H*| alone (distributions + subset selection, no convex solve): usable on
    supports far too large for the solvers."""
    tl, dl = _f64(tl), _f64(dl)
    V = tl.shape[0]
    tgt, drf, ids, _ = distributions(tl, dl, topk, Tt, Td)
    k = ids.shape[0]
    ids = _i32(ids)
    order = np.empty(k, dtype=np.int32)
    psi = np.empty(k + 1); Tg = np.empty(k + 1); Dr = np.empty(k + 1)
    a = C.c_double(0)
    D = C.c_double
    js = lib().gro_subset_selection(_p(tl, D), _p(dl, D), _p(tgt, D), _p(drf, D), _p(ids, C.c_int), k, int(n),
                                    D(Tt), D(Td), int(k == V), _p(order, C.c_int), _p(psi, D), _p(Tg, D), _p(Dr, D),
                                    C.byref(a))
    return a.value, int(js)


def grad(route, d, w, n, h=0.0, slack=True):
    d, w = _f64(d), _f64(w)
    m = d.shape[0]
    g = np.zeros(m)
    fn = lib().gro_grad_g1 if route == ROUTE_G1 else lib().gro_grad_g2
    st = fn(m, _p(d, C.c_double), _p(w, C.c_double), int(n), C.c_double(h), int(bool(slack)), _p(g, C.c_double))
    if st < 0:
        raise ValueError("bad argument")
    return g


def fit(route, d, rhs, n, h=0.0, slack=True, tol=1e-12, max_iter=2000, method=METHOD_NEWTON):
    d, rhs = _f64(d), _f64(rhs)
    m = d.shape[0]
    w = np.ones(m)
    gn = C.c_double(0)
    it = C.c_int(0)
    fn = lib().gro_ipf if method == METHOD_IPF else lib().gro_newton
    st = fn(int(route), m, _p(d, C.c_double), _p(rhs, C.c_double), int(n), C.c_double(h),
                       int(bool(slack)), C.c_double(tol), int(max_iter), _p(w, C.c_double), C.byref(gn), C.byref(it))
    return w, gn.value, it.value, st


@dataclasses.dataclass
class Solution:
    V: int
    n: int
    k: int
    jstar: int
    nblocks: int
    alpha_star: float
    order: np.ndarray      # [k] token id at each ratio-order position
    tgt_pos: np.ndarray    # [k]
    drf_pos: np.ndarray    # [k]
    psi: np.ndarray        # [k+1]
    p: np.ndarray          # [k]  flow each support token receives from tuples (tgt on H*)
    r: np.ndarray          # [k]  residual of each support token (0 on H*)
    block: np.ndarray      # [k]  -1 on H*, else block number from the lowest ratio
    w: np.ndarray          # [k]  exp(alpha)
    gnorm: float
    iters: int
    status: int
    tgt_full: np.ndarray   # [V]
    drf_full: np.ndarray   # [V]

    def residual_full(self) -> np.ndarray:
        r = self.tgt_full.copy()
        r[self.order] = self.r
        return r


def solve(tl, dl, n, topk, Tt=1.0, Td=1.0, route=ROUTE_G2, tol=1e-12, max_iter=2000,
          method=METHOD_NEWTON, tau=0.0) -> Solution:
    tl, dl = _f64(tl), _f64(dl)
    V = tl.shape[0]
    kmax = V if (topk <= 0 or topk >= V) else topk
    tgt = np.empty(V); drf = np.empty(V)
    order = np.empty(kmax, dtype=np.int32); block = np.empty(kmax, dtype=np.int32)
    tgt_pos = np.empty(kmax); drf_pos = np.empty(kmax); psi = np.empty(kmax + 1)
    p = np.empty(kmax); r = np.empty(kmax); w = np.ones(kmax)
    k = C.c_int(0); jstar = C.c_int(0); nb = C.c_int(0); it = C.c_int(0)
    a = C.c_double(0); gn = C.c_double(0)
    D = C.c_double
    st = lib().gro_solve(_p(tl, D), _p(dl, D), V, int(n), int(topk), D(Tt), D(Td), int(route), int(method), D(tol), int(max_iter),
                         D(tau), _p(tgt, D), _p(drf, D), C.byref(k), _p(order, C.c_int), _p(tgt_pos, D), _p(drf_pos, D),
                         _p(psi, D), C.byref(jstar), C.byref(a), _p(p, D), _p(r, D), _p(block, C.c_int),
                         C.byref(nb), _p(w, D), C.byref(gn), C.byref(it))
    if st < 0:
        raise ValueError("bad argument")
    return Solution(V, n, k.value, jstar.value, nb.value, a.value, order, tgt_pos, drf_pos, psi, p, r, block, w,
                    gn.value, it.value, st, tgt, drf)


def slice_(sol: Solution, omega):
    omega = _i32(omega)
    n = omega.shape[0]
    U = np.full(n, -1, dtype=np.int32)
    pi = np.zeros(n)
    rho = C.c_double(0)
    nu = lib().gro_slice(sol.k, n, sol.jstar, _p(sol.order, C.c_int), _p(sol.block, C.c_int),
                         _p(_f64(sol.w), C.c_double), _p(omega, C.c_int), _p(U, C.c_int), _p(pi, C.c_double),
                         C.byref(rho))
    if nu < 0:
        return nu, None, None, None
    return nu, U[:nu].copy(), pi[:nu].copy(), rho.value


def draw(U, pi, rho, r_full, u0, u1):
    U = _i32(U); pi = _f64(pi); r_full = _f64(r_full)
    tok = C.c_int(-1); acc = C.c_int(0)
    lib().gro_draw(U.shape[0], _p(U, C.c_int), _p(pi, C.c_double), C.c_double(rho), _p(r_full, C.c_double),
                   r_full.shape[0], C.c_double(float(u0)), C.c_double(float(u1)), C.byref(tok), C.byref(acc))
    return tok.value, acc.value


@dataclasses.dataclass
class BatchResult:
    alpha_star: np.ndarray
    token: np.ndarray
    accepted: np.ndarray
    status: np.ndarray
    U: np.ndarray        # [B, n] distinct drafted ids in first-occurrence order, -1 padded
    pi: np.ndarray       # [B, n]
    rho: np.ndarray      # [B]
    gnorm: np.ndarray
    iters: np.ndarray
    jstar: np.ndarray
    # the whole solution of every instance, per-support arrays [B, kcap] in ratio order (padding -1 / -2 / 0)
    k: np.ndarray
    nblocks: np.ndarray
    order: np.ndarray
    block: np.ndarray
    w: np.ndarray
    r: np.ndarray
    p: np.ndarray
    psi: np.ndarray      # [B, kcap + 1]


def solve_verify_batch(tl, dl, n, topk, Tt, Td, draft_tokens, uniforms, route=ROUTE_G2, tol=1e-12,
                       max_iter=2000, method=METHOD_NEWTON, tau=0.0) -> BatchResult:
    tl, dl = _f64(tl), _f64(dl)
    B, V = tl.shape
    toks = _i32(draft_tokens); uni = np.ascontiguousarray(uniforms, dtype=np.float32)
    assert toks.shape == (B, n) and uni.shape == (B, 2)
    a = np.zeros(B); token = np.zeros(B, dtype=np.int32); acc = np.zeros(B, dtype=np.int32)
    status = np.zeros(B, dtype=np.int32); U = np.zeros((B, n), dtype=np.int32); pi = np.zeros((B, n))
    rho = np.zeros(B); gn = np.zeros(B); it = np.zeros(B, dtype=np.int32); js = np.zeros(B, dtype=np.int32)
    kcap = V if (topk <= 0 or topk >= V) else int(topk)
    kk = np.zeros(B, dtype=np.int32); nb = np.zeros(B, dtype=np.int32)
    order = np.zeros((B, kcap), dtype=np.int32); block = np.zeros((B, kcap), dtype=np.int32)
    w = np.zeros((B, kcap)); r = np.zeros((B, kcap)); p = np.zeros((B, kcap)); psi = np.zeros((B, kcap + 1))
    D = C.c_double
    lib().gro_solve_verify_batch(_p(tl, D), _p(dl, D), B, V, int(n), int(topk), D(Tt), D(Td), int(route), int(method), D(tol),
                                 int(max_iter), D(tau), _p(toks, C.c_int), _p(uni, C.c_float), _p(a, D), _p(token, C.c_int),
                                 _p(acc, C.c_int), _p(status, C.c_int), _p(U, C.c_int), _p(pi, D), _p(rho, D),
                                 _p(gn, D), _p(it, C.c_int), _p(js, C.c_int),
                                 kcap, _p(kk, C.c_int), _p(nb, C.c_int), _p(order, C.c_int), _p(block, C.c_int),
                                 _p(w, D), _p(r, D), _p(p, D), _p(psi, D))
    return BatchResult(a, token, acc, status, U, pi, rho, gn, it, js, kk, nb, order, block, w, r, p, psi)


@dataclasses.dataclass
class Certificate:
    k: np.ndarray
    jstar: np.ndarray
    nblocks: np.ndarray
    alpha_star: np.ndarray
    order: np.ndarray    # [B, kcap] token ids in ratio order, -1 padded
    block: np.ndarray    # [B, kcap]
    r: np.ndarray
    p: np.ndarray
    psi: np.ndarray      # [B, kcap + 1]
    gnorm: np.ndarray    # [B] L1 gradient norm of the convex functions at the given weights
    gnorm_lse: np.ndarray  # [B] the same with the target normalised by the log-sum-exp given from outside (nan if none)
    lse_target: np.ndarray  # [B] the oracle's own log-sum-exp of the target row


def certify_batch(tl, dl, n, topk, Tt, Td, w, lse=None) -> Certificate:
    """Structure of every instance (no solve) and the L1 gradient norm at weights given from outside
    ([B, kcap] in ratio order): one gradient evaluation per system.  `lse` ([B], optional): a target
    log-sum-exp from outside; gnorm_lse is then the norm with the target normalised by it."""
    tl, dl = _f64(tl), _f64(dl)
    B, V = tl.shape
    w = _f64(w)
    kcap = w.shape[1]
    kk = np.zeros(B, dtype=np.int32); js = np.zeros(B, dtype=np.int32); nb = np.zeros(B, dtype=np.int32)
    a = np.zeros(B); cert = np.zeros(B)
    order = np.zeros((B, kcap), dtype=np.int32); block = np.zeros((B, kcap), dtype=np.int32)
    r = np.zeros((B, kcap)); p = np.zeros((B, kcap)); psi = np.zeros((B, kcap + 1))
    D = C.c_double
    cert2 = np.full(B, np.nan); lse_own = np.zeros(B)
    lse_arr = _f64(lse) if lse is not None else None
    st = lib().gro_certify_batch(_p(tl, D), _p(dl, D), B, V, int(n), int(topk), D(Tt), D(Td), _p(w, D), kcap,
                                 _p(lse_arr, D) if lse_arr is not None else None,
                                 _p(cert2, D) if lse_arr is not None else None, _p(lse_own, D),
                                 _p(kk, C.c_int), _p(js, C.c_int), _p(nb, C.c_int), _p(a, D), _p(order, C.c_int),
                                 _p(block, C.c_int), _p(r, D), _p(p, D), _p(psi, D), _p(cert, D))
    if st < 0:
        raise ValueError("bad argument")
    return Certificate(kk, js, nb, a, order, block, r, p, psi, cert, cert2, lse_own)


def draw_sweep_batch(tl, dl, n, topk, Tt, Td, res: BatchResult, draft_tokens, uniforms):
    """R draws per instance from the rules in `res` (uniforms [B, R, 2]): tokens [B, R], accepted [B, R] and the
    distance of the deciding uniform to the nearest CDF boundary [B, R]."""
    tl, dl = _f64(tl), _f64(dl)
    B, V = tl.shape
    toks = _i32(draft_tokens)
    uni = np.ascontiguousarray(uniforms, dtype=np.float32)
    R = uni.shape[1]
    assert uni.shape == (B, R, 2) and toks.shape == (B, n)
    kcap = res.order.shape[1]
    token = np.zeros((B, R), dtype=np.int32); acc = np.zeros((B, R), dtype=np.int32); margin = np.zeros((B, R))
    D = C.c_double
    lib().gro_draw_sweep_batch(_p(tl, D), _p(dl, D), B, V, int(n), int(topk), D(Tt), D(Td), kcap,
                               _p(_i32(res.k), C.c_int), _p(_i32(res.jstar), C.c_int), _p(_i32(res.order), C.c_int),
                               _p(_i32(res.block), C.c_int), _p(_f64(res.w), D), _p(_f64(res.r), D),
                               _p(toks, C.c_int), _p(uni, C.c_float), R, _p(token, C.c_int), _p(acc, C.c_int),
                               _p(margin, D))
    return token, acc, margin


def truncation_sets(order, drf_pos, jstar, n, tau):
    """Minimal truncation sets (Sec. 6.2-6.3): (in_T [k] of 0/1 in ratio order, gamma_T, epsilon_T)."""
    order = _i32(order); d = _f64(drf_pos)
    k = d.shape[0]
    in_T = np.zeros(k, dtype=np.int32)
    gam = C.c_double(0); eps = C.c_double(0)
    lib().gro_truncation_sets(k, int(jstar), _p(order, C.c_int), _p(d, C.c_double), int(n), C.c_double(tau),
                              _p(in_T, C.c_int), C.byref(gam), C.byref(eps))
    return in_T, gam.value, eps.value


def rule_deviation(sol: Solution, w=None):
    """(L1 distance of the emitted-token marginal from the target, acceptance, flows [k]) of the rule that the
    structure of `sol` and the weights `w` (default: its own; zeros allowed) define."""
    k = sol.k
    w = _f64(sol.w[:k] if w is None else w)
    l1 = C.c_double(0); acc = C.c_double(0)
    flow = np.zeros(max(k, 1))
    D = C.c_double
    lib().gro_rule_deviation(k, int(sol.n), int(sol.jstar), int(sol.nblocks), _p(_i32(sol.block[:k]), C.c_int),
                             _p(_f64(sol.tgt_pos[:k]), D), _p(_f64(sol.drf_pos[:k]), D), _p(_f64(sol.r[:k]), D),
                             _p(w, D), D(sol.alpha_star), C.byref(l1), C.byref(acc), _p(flow, D))
    return l1.value, acc.value, flow[:k]


def num_threads() -> int:
    return int(lib().gro_num_threads())
