"""Exponential-size reference computations used to pin the oracle (numpy / scipy only).

Everything here works from the definitions: the relaxed transport LP over all
V^n draft tuples, the max-flow network, subset enumeration, tuple enumeration of
the softmax row sums.  None of it calls the oracle.
"""
import itertools

import numpy as np
import scipy.optimize
import scipy.sparse
import scipy.sparse.csgraph


def tuples(V, n):
    return list(itertools.product(range(V), repeat=n))


def draft_tuple_prob(drf, om):
    pr = 1.0
    for s in om:
        pr *= drf[s]
    return pr


def relaxed_otlp_value(tgt, drf, n):
    """max sum S  s.t. row sums <= tgt, column sums <= drf^n(omega), S_{i,omega}=0 unless i in set(omega)
    (Eq. relaxed-lp), solved with HiGHS."""
    V = len(tgt)
    toms = tuples(V, n)
    var = []
    for c, om in enumerate(toms):
        for i in sorted(set(om)):
            var.append((i, c))
    nv = len(var)
    rows, cols = [], []
    for v, (i, c) in enumerate(var):
        rows.append(i); cols.append(v)
        rows.append(V + c); cols.append(v)
    A = scipy.sparse.csr_matrix((np.ones(len(rows)), (rows, cols)), shape=(V + len(toms), nv))
    b = np.concatenate([tgt, [draft_tuple_prob(drf, om) for om in toms]])
    res = scipy.optimize.linprog(-np.ones(nv), A_ub=A, b_ub=b, bounds=(0, None), method="highs")
    assert res.status == 0
    return -res.fun


def maxflow_value_int(tgt_int, drf_int, n):
    """Max-flow on the network s -> i (cap tgt_i) -> omega (cap inf, i in set(omega)) -> t (cap drf^n(omega))
    (Sec. 5.2) with integer capacities: tgt_int_i and prod_s drf_int[omega_s]."""
    V = len(tgt_int)
    toms = tuples(V, n)
    N = 2 + V + len(toms)
    s, t = 0, 1
    r, c, cap = [], [], []
    big = int(sum(tgt_int)) + 1
    for i in range(V):
        r.append(s); c.append(2 + i); cap.append(int(tgt_int[i]))
    for j, om in enumerate(toms):
        node = 2 + V + j
        pr = 1
        for x in om:
            pr *= int(drf_int[x])
        r.append(node); c.append(t); cap.append(pr)
        for i in set(om):
            r.append(2 + i); c.append(node); cap.append(big)
    g = scipy.sparse.csr_matrix((np.array(cap, dtype=np.int64), (r, c)), shape=(N, N))
    return scipy.sparse.csgraph.maximum_flow(g.astype(np.int64), s, t).flow_value


def psi(tgt, drf, n, mask):
    return tgt[mask].sum() - drf[mask].sum() ** n


def all_subset_psi(tgt, drf, n):
    """psi(H) for every H (bitmask index), vectorised."""
    V = len(tgt)
    masks = np.arange(1 << V, dtype=np.int64)
    bits = ((masks[:, None] >> np.arange(V)[None, :]) & 1).astype(np.float64)
    return bits @ tgt - (bits @ drf) ** n


def inner_rowsums_enum(w, d, n):
    """sum over omega in support^n of drf^n(omega) w_i/(1+sum_{set} w)  (Eq. defined-s-inner summed)."""
    k = len(w)
    g = np.zeros(k)
    for om in tuples(k, n):
        pr = draft_tuple_prob(d, om)
        S = set(om)
        W = 1.0 + sum(w[j] for j in S)
        for i in S:
            g[i] += pr * w[i] / W
    return g


def outer_rowsums_enum(w, d, n, h):
    """Block members 0..m-1 plus one lumped higher-ratio symbol of mass h (index m) that takes no flow:
    sum over tuples touching the block of drf^n(omega) w_i / sum_{set n block} w  (Eq. defined-s-outer summed)."""
    m = len(w)
    dd = np.concatenate([d, [h]])
    g = np.zeros(m)
    for om in tuples(m + 1, n):
        S = set(om) - {m}
        if not S:
            continue
        pr = draft_tuple_prob(dd, om)
        W = sum(w[j] for j in S)
        for i in S:
            g[i] += pr * w[i] / W
    return g
