"""Pins of the oracle's integral gradient route at the support sizes and draft counts the GPU is compared on.

The integral route (gro_grad_g2) is the only gradient evaluation that reaches supports of 50 or 100
tokens with 8 to 32 drafts, so it is pinned there against things that are not the integral:
  - an exact closed form for supports made of a few groups of identical tokens (the grouped-term
    weights of App. K collapse by symmetry to a sum over group counts; evaluated in integer / rational
    arithmetic, so there is no rounding or cancellation in the reference);
  - enumeration of all draft tuples straight from the definition of the row sums (Eqs.
    "defined-s-inner" / "defined-s-outer") at 50 tokens with 2 and 3 drafts and at 8 tokens with 8 drafts;
  - the grouped-term route at n = 32 on small supports;
  - the total flow of an outer block (mass of the tuples it serves), which holds for any weights;
  - seeded sampling of draft tuples from the definition (statistical, 5 sigma) at (50, 8) and (100, 16).
"""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import gr_oracle as O


# ---------------------------------------------------------------- exact closed form on grouped supports

def _transform_axis(X, axis):
    """T[s] = sum_j (-1)^(s-j) C(s, j) X[j] along one axis of an object array of Python ints."""
    X = np.moveaxis(X, axis, 0)
    S = X.shape[0]
    out = np.empty_like(X)
    for s in range(S):
        acc = 0
        for j in range(s + 1):
            term = math.comb(s, j) * X[j]
            acc = acc + term if (s - j) % 2 == 0 else acc - term
        out[s] = acc
    return np.moveaxis(out, 0, axis)


def _grouped_rowsums_exact(sizes, dnum, D, hnum, wfrac, n, slack):
    """Exact row sums for a support of len(sizes) groups: group g has sizes[g] tokens of draft mass
    dnum[g] / D and weight wfrac[g]; hnum / D is the mass of the higher-ratio symbol (outer block) or 0.

    A set A with s_g tokens of group g is the exact set of distinct block tokens of a tuple with probability
      sum_{j <= s} prod_g (-1)^(s_g - j_g) C(s_g, j_g) (h + sum_g j_g d_g)^n        (App. K),
    and a token of group a belongs to C(m_a - 1, s_a - 1) prod_{g != a} C(m_g, s_g) such sets, in each of
    which it receives the share w_a / (slack + sum_g s_g w_g)."""
    G = len(sizes)
    caps = [min(n, m) for m in sizes]
    shape = tuple(c + 1 for c in caps)
    X = np.empty(shape, dtype=object)
    for j in itertools.product(*[range(c + 1) for c in caps]):
        X[j] = (hnum + sum(jg * dg for jg, dg in zip(j, dnum))) ** n
    for ax in range(G):
        X = _transform_axis(X, ax)
    denom = D ** n
    out = []
    for a in range(G):
        tot = Fraction(0)
        for s in itertools.product(*[range(c + 1) for c in caps]):
            if s[a] == 0 or sum(s) > n or X[s] == 0:
                continue
            cnt = math.comb(sizes[a] - 1, s[a] - 1)
            for g in range(G):
                if g != a:
                    cnt *= math.comb(sizes[g], s[g])
            Wt = (1 if slack else 0) + sum(sg * wg for sg, wg in zip(s, wfrac))
            tot += Fraction(cnt * X[s], denom) * wfrac[a] / Wt
        out.append(tot)
    return out


GROUPED = [
    # sizes, draft numerators, common denominator, weights, n
    ((3, 12, 35), (40, 10, 2), 400, (Fraction(3, 1000), Fraction(7, 2), Fraction(120000)), 8),          # 50 tokens
    ((2, 8, 40), (90, 15, 4), 800, (Fraction(25000), Fraction(1, 500), Fraction(9, 4)), 8),             # 50 tokens
    ((4, 26, 70), (60, 10, 3), 1000, (Fraction(11, 10), Fraction(40000), Fraction(1, 250)), 16),        # 100 tokens
    ((6, 18), (50, 10), 600, (Fraction(2, 1000), Fraction(31000)), 32),                                 # 24 tokens
    ((1, 19), (400, 20), 800, (Fraction(5), Fraction(1, 3)), 32),                                       # one dominant token
]


@pytest.mark.parametrize("sizes,dnum,D,wfrac,n", GROUPED)
def test_integral_route_equals_exact_grouped_closed_form(sizes, dnum, D, wfrac, n):
    total = sum(m * d for m, d in zip(sizes, dnum))
    d = np.concatenate([np.full(m, dg / D) for m, dg in zip(sizes, dnum)])
    w = np.concatenate([np.full(m, float(wg)) for m, wg in zip(sizes, wfrac)])
    starts = np.cumsum([0] + list(sizes[:-1]))
    # inner system: the support carries all the draft mass it has (total / D <= 1), slack vertex of weight 1
    assert total <= D
    exact = _grouped_rowsums_exact(sizes, dnum, D, 0, wfrac, n, True)
    g = O.grad(O.ROUTE_G2, d, w, n)
    for a, s0 in enumerate(starts):
        ref = float(exact[a])
        assert np.allclose(g[s0:s0 + sizes[a]], ref, rtol=2e-10, atol=1e-14), (a, g[s0], ref)
    # outer block: the rest of the mass sits on a higher-ratio symbol that takes no flow
    hnum = D - total
    exact_o = _grouped_rowsums_exact(sizes, dnum, D, hnum, wfrac, n, False)
    go = O.grad(O.ROUTE_G2, d, w, n, h=hnum / D, slack=False)
    for a, s0 in enumerate(starts):
        ref = float(exact_o[a])
        assert np.allclose(go[s0:s0 + sizes[a]], ref, rtol=2e-10, atol=1e-14), (a, go[s0], ref)
    flow = float(sum(m * e for m, e in zip(sizes, exact_o)))
    assert abs(flow - (1.0 - (hnum / D) ** n)) < 1e-12


# ---------------------------------------------------------------- tuple enumeration from the definition

def _rowsums_by_enumeration(d, w, n, h, slack):
    """All tuples over the support (plus, for an outer block, one symbol of mass h that takes no flow)."""
    m = len(d)
    if h > 0:
        dd = np.concatenate([d, [h]]); ww = np.concatenate([w, [0.0]])
    else:
        dd, ww = d, w
    M = len(dd)
    idx = np.stack(np.meshgrid(*[np.arange(M)] * n, indexing="ij"), axis=-1).reshape(-1, n)
    pr = np.prod(dd[idx], axis=1)
    first = np.ones(idx.shape, dtype=bool)
    for s in range(1, n):
        for s2 in range(s):
            first[:, s] &= idx[:, s] != idx[:, s2]
    Wt = (1.0 if slack else 0.0) + np.sum(np.where(first, ww[idx], 0.0), axis=1)
    g = np.zeros(M)
    for s in range(n):
        ok = first[:, s] & (Wt > 0)
        np.add.at(g, idx[ok, s], pr[ok] * ww[idx[ok, s]] / Wt[ok])
    return g[:m]


@pytest.mark.parametrize("n", [2, 3])
def test_integral_route_equals_tuple_enumeration_at_50_tokens(n):
    rng = np.random.default_rng(50 + n)
    m = 50
    d = rng.dirichlet(0.4 * np.ones(m))
    w = np.exp(rng.uniform(np.log(1e-3), np.log(1e5), m))
    ref = _rowsums_by_enumeration(d, w, n, 0.0, True)
    assert np.allclose(O.grad(O.ROUTE_G2, d, w, n), ref, rtol=1e-10, atol=1e-15)
    ref_o = _rowsums_by_enumeration(0.7 * d, w, n, 0.3, False)
    assert np.allclose(O.grad(O.ROUTE_G2, 0.7 * d, w, n, h=0.3, slack=False), ref_o, rtol=1e-10, atol=1e-15)


def test_integral_route_equals_tuple_enumeration_at_8_tokens_8_drafts():
    """8^8 = 1.7e7 tuples, grouped by their set of distinct tokens (a bitmask) as they are enumerated."""
    rng = np.random.default_rng(88)
    m, n = 8, 8
    d = rng.dirichlet(0.6 * np.ones(m))
    w = np.exp(rng.uniform(np.log(1e-2), np.log(1e4), m))
    mass = np.zeros(1 << m)
    # enumerate the first four and the last four drafts separately and combine their (mask, probability) tables
    half = np.stack(np.meshgrid(*[np.arange(m)] * 4, indexing="ij"), axis=-1).reshape(-1, 4)
    hmask = np.bitwise_or.reduce(1 << half, axis=1)
    hpr = np.prod(d[half], axis=1)
    tab = np.bincount(hmask, weights=hpr, minlength=1 << m)        # Pr[first four drafts cover exactly this set]
    for a in np.nonzero(tab)[0]:
        for b in np.nonzero(tab)[0]:
            mass[a | b] += tab[a] * tab[b]
    assert abs(mass.sum() - 1.0) < 1e-13
    g = np.zeros(m)
    for A in range(1, 1 << m):
        members = [j for j in range(m) if A >> j & 1]
        Wt = 1.0 + w[members].sum()
        g[members] += mass[A] * w[members] / Wt
    assert np.allclose(O.grad(O.ROUTE_G2, d, w, n), g, rtol=1e-10, atol=1e-15)


# ---------------------------------------------------------------- the two routes at n = 32

@pytest.mark.parametrize("m", [6, 10, 12])
def test_integral_route_equals_grouped_terms_at_32_drafts(m):
    rng = np.random.default_rng(3200 + m)
    d = rng.dirichlet(0.5 * np.ones(m))
    d[0] += 0.6; d /= d.sum()                    # one dominant draft token, as in the n = 32 workloads
    w = np.exp(rng.normal(0, 3.0, m))
    g1 = O.grad(O.ROUTE_G1, d, w, 32)
    g2 = O.grad(O.ROUTE_G2, d, w, 32)
    assert np.allclose(g1, g2, rtol=1e-8, atol=1e-12)
    g1o = O.grad(O.ROUTE_G1, 0.5 * d, w, 32, h=0.5, slack=False)
    g2o = O.grad(O.ROUTE_G2, 0.5 * d, w, 32, h=0.5, slack=False)
    assert np.allclose(g1o, g2o, rtol=1e-8, atol=1e-12)


# ---------------------------------------------------------------- invariants at full size

@pytest.mark.parametrize("m,n", [(50, 8), (100, 16), (20, 32), (128, 16)])
def test_outer_block_total_flow_for_arbitrary_weights(m, n):
    """sum_i g_i = (h + sum d)^n - h^n whatever the weights: every tuple touching the block gives it all its mass."""
    rng = np.random.default_rng(m * 100 + n)
    for h in (0.0, 0.35):
        d = rng.dirichlet(0.5 * np.ones(m)) * (1.0 - h)
        w = np.exp(rng.uniform(np.log(1e-3), np.log(1e5), m))
        g = O.grad(O.ROUTE_G2, d, w, n, h=h, slack=False)
        assert np.all(g > 0)
        assert abs(g.sum() - (1.0 - h ** n)) < 1e-11
        # inner system: flows grow with a common scale of the weights and tend to the outer block's as the slack vanishes
        gi = O.grad(O.ROUTE_G2, d, w, n)
        gi2 = O.grad(O.ROUTE_G2, d, 4.0 * w, n)
        assert np.all(gi2 > gi) and gi2.sum() < (1.0 - h) ** n + 1e-12
    d = rng.dirichlet(0.5 * np.ones(m))
    w = np.exp(rng.uniform(np.log(1e-1), np.log(1e2), m))
    lim = O.grad(O.ROUTE_G2, d, w, n, h=0.0, slack=False)
    big = O.grad(O.ROUTE_G2, d, 1e9 * w, n)
    assert np.allclose(big, lim, rtol=1e-6, atol=1e-12)


# ---------------------------------------------------------------- sampling the definition

@pytest.mark.parametrize("m,n,N", [(50, 8, 400000), (100, 16, 250000)])
def test_integral_route_within_sampling_error_of_the_definition(m, n, N):
    """Draft tuples drawn i.i.d. from drf; each distinct drafted token i receives w_i / (1 + sum over the distinct
    drafted tokens of w).  The mean over tuples estimates the row sum; its standard error is estimated from the
    same sample."""
    rng = np.random.default_rng(m * 1000 + n)
    ranks = np.arange(1, m + 1)
    d = (1.0 / ranks) * np.exp(rng.normal(0, 0.5, m)); d /= d.sum()
    w = np.exp(rng.uniform(np.log(1e-2), np.log(3e4), m))
    cdf = np.cumsum(d)
    s1 = np.zeros(m); s2 = np.zeros(m)
    chunk = 50000
    for c0 in range(0, N, chunk):
        om = np.searchsorted(cdf, rng.random((min(chunk, N - c0), n)) * cdf[-1], side="right").clip(max=m - 1)
        om.sort(axis=1)
        first = np.ones(om.shape, dtype=bool)
        first[:, 1:] = om[:, 1:] != om[:, :-1]
        Wt = 1.0 + np.sum(np.where(first, w[om], 0.0), axis=1)
        share = np.where(first, w[om] / Wt[:, None], 0.0)
        s1 += np.bincount(om[first], weights=share[first], minlength=m)
        s2 += np.bincount(om[first], weights=share[first] ** 2, minlength=m)
    mean = s1 / N
    sigma = np.sqrt(np.maximum(s2 / N - mean ** 2, 0.0) / N)
    g = O.grad(O.ROUTE_G2, d, w, n)
    z = np.abs(g - mean) / (sigma + 1e-12)
    assert np.all(z < 5.0), (float(z.max()), int(np.argmax(z)))
    assert abs(g.sum() - mean.sum()) < 5.0 * np.sqrt((sigma ** 2).sum()) + 1e-9
