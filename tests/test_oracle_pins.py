"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these retype the oracle's formulas: they compare it with exponential-size
definitions (LP / max-flow over all V^n tuples, 2^V subset enumeration, tuple
enumeration), closed forms (n = 1) and invariants (Hall inequalities, marginals).
"""
import itertools

import numpy as np
import pytest

from oracle import gr_oracle as O
from paper_2511_15898_b200 import workloads as W
from tests import bruteforce as BF


def _rand_logits(rng, V, scale=2.0, dnoise=0.7):
    tl = scale * rng.standard_normal(V)
    dl = tl + dnoise * rng.standard_normal(V)
    return tl, dl


# ---------------------------------------------------------------- alpha*  (Eq. subset-select, Sec. 5.1-5.2)

@pytest.mark.parametrize("V,n,topk", [(4, 2, 0), (5, 3, 0), (6, 2, 3), (5, 3, 3), (7, 2, 0)])
def test_alpha_star_equals_relaxed_lp(V, n, topk):
    rng = np.random.default_rng(100 * V + 10 * n + topk)
    for _ in range(4):
        tl, dl = _rand_logits(rng, V)
        sol = O.solve(tl, dl, n, topk, route=O.ROUTE_G1, tol=1e-9)
        lp = BF.relaxed_otlp_value(sol.tgt_full, sol.drf_full, n)
        assert abs(sol.alpha_star - lp) < 1e-8
        # the drafts never leave the kept ids, so the LP on the kept slice is the same problem (App. N)
        if topk:
            ids = np.sort(sol.order)
            lp2 = BF.relaxed_otlp_value(sol.tgt_full[ids], sol.drf_full[ids], n)
            assert abs(lp - lp2) < 1e-8


def test_alpha_star_equals_integer_maxflow():
    """Dyadic probabilities make every capacity an integer, so max-flow is exact."""
    rng = np.random.default_rng(7)
    for V, n, bits_d in [(5, 2, 5), (4, 3, 4), (6, 2, 6)]:
        for _ in range(3):
            D = 1 << bits_d
            dcounts = rng.multinomial(D - V, np.ones(V) / V) + 1            # sums to 2^bits_d
            T = D ** n
            tcounts = rng.multinomial(T - V, rng.dirichlet(np.ones(V))) + 1  # sums to 2^(bits_d*n)
            tl = np.log(tcounts.astype(np.float64))
            dl = np.log(dcounts.astype(np.float64))
            sol = O.solve(tl, dl, n, 0, route=O.ROUTE_G1, tol=1e-9)
            mf = BF.maxflow_value_int(tcounts, dcounts, n)
            assert abs(sol.alpha_star - mf / T) < 1e-12


@pytest.mark.parametrize("n", [1, 2, 3, 5, 8])
def test_alpha_star_equals_subset_enumeration(n):
    rng = np.random.default_rng(n)
    for V, topk in [(8, 0), (10, 4), (12, 0)]:
        tl, dl = _rand_logits(rng, V)
        tgt, drf, ids, _ = O.distributions(tl, dl, topk, 1.0, 1.0)
        sol = O.solve(tl, dl, n, topk, tol=1e-9)
        allpsi = BF.all_subset_psi(tgt, drf, n)
        assert abs(sol.alpha_star - (1.0 + allpsi.min())) < 1e-13
        # H* is the smallest minimiser
        mask = 0
        for t in sol.order[: sol.jstar]:
            mask |= 1 << int(t)
        assert abs(allpsi[mask] - allpsi.min()) < 1e-13


def test_config1_alpha_star_subset_enumeration():
    wl = W.config1(batch=8)
    tl = W.logits_to_f64(wl.q_logits); dl = W.logits_to_f64(wl.p_logits)
    for b in range(8):
        sol = O.solve(tl[b], dl[b], wl.n, wl.topk, tol=1e-9)
        allpsi = BF.all_subset_psi(sol.tgt_full, sol.drf_full, wl.n)
        assert abs(sol.alpha_star - (1.0 + allpsi.min())) < 1e-13


def test_n1_reduces_to_single_draft_speculative_sampling():
    """n = 1: alpha* = sum_x min(tgt, drf); acceptance of x is min(1, tgt/drf); resample ~ (tgt-drf)+."""
    rng = np.random.default_rng(11)
    V = 9
    tl, dl = _rand_logits(rng, V)
    sol = O.solve(tl, dl, 1, 0, tol=1e-13)
    tgt, drf = sol.tgt_full, sol.drf_full
    assert abs(sol.alpha_star - np.minimum(tgt, drf).sum()) < 1e-14
    res = np.maximum(tgt - drf, 0.0)
    assert np.allclose(sol.residual_full(), res, atol=1e-14)
    for x in range(V):
        nu, U, pi, rho = O.slice_(sol, [x])
        assert nu == 1 and U[0] == x
        assert abs(pi[0] - min(1.0, tgt[x] / drf[x])) < 1e-10
        assert abs(pi[0] + rho - 1.0) < 1e-12


def test_alpha_star_monotone_in_n_and_at_most_one():
    rng = np.random.default_rng(5)
    tl, dl = _rand_logits(rng, 40, dnoise=1.5)
    prev = -1.0
    for n in [1, 2, 3, 4, 6, 8, 16, 32]:
        a = O.solve(tl, dl, n, 10, tol=1e-6, max_iter=50).alpha_star
        assert a <= 1.0 + 1e-15
        assert a >= prev - 1e-15
        prev = a


def test_temperature_and_topk_only_change_the_distributions():
    rng = np.random.default_rng(3)
    tl, dl = _rand_logits(rng, 30)
    tgt, drf, ids, lse = O.distributions(tl, dl, 7, 0.7, 1.3)
    e = np.exp(tl / 0.7 - np.max(tl / 0.7)); assert np.allclose(tgt, e / e.sum(), atol=1e-15)
    top = np.argsort(-dl, kind="stable")[:7]
    assert sorted(top.tolist()) == ids.tolist()
    ed = np.exp(dl[top] / 1.3); ref = np.zeros(30); ref[top] = ed / ed.sum()
    assert np.allclose(drf, ref, atol=1e-15)
    # ties at the cut: the smaller id is kept
    dl2 = np.array([0.0, 1.0, 1.0, 1.0, -1.0]); tl2 = np.zeros(5)
    _, drf2, ids2, _ = O.distributions(tl2, dl2, 2, 1.0, 1.0)
    assert ids2.tolist() == [1, 2]


# ---------------------------------------------------------------- outer residuals (Sec. 6.1)

def _outer_cases():
    rng = np.random.default_rng(21)
    cases = []
    for V, n, topk in [(7, 2, 0), (8, 3, 0), (8, 2, 5), (9, 4, 6), (10, 2, 0)]:
        for _ in range(3):
            tl = 1.5 * rng.standard_normal(V)
            dl = tl + 1.2 * rng.standard_normal(V)
            cases.append((tl, dl, n, topk))
    return cases


def test_outer_residuals_match_theorem_by_superset_enumeration():
    """p_v = tgt(v) + min_{T >= H_{i+1}} psi(T) - min_{T >= H_i} psi(T), minima by brute force over all T."""
    seen_outer = 0
    for tl, dl, n, topk in _outer_cases():
        sol = O.solve(tl, dl, n, topk, tol=1e-6, max_iter=10)
        V = sol.V
        allpsi = BF.all_subset_psi(sol.tgt_full, sol.drf_full, n)
        masks = np.arange(1 << V)

        def min_over_supersets(hmask):
            return allpsi[(masks & hmask) == hmask].min()

        hstar = 0
        for t in sol.order[: sol.jstar]:
            hstar |= 1 << int(t)
        # chain in increasing ratio: zero-draft ids first (any order), then support positions k-1 .. jstar
        zero_ids = [i for i in range(V) if sol.drf_full[i] == 0.0]
        chain = zero_ids + [int(sol.order[pos]) for pos in range(sol.k - 1, sol.jstar - 1, -1)]
        rfull = sol.residual_full()
        for i, v in enumerate(chain):
            Hi = hstar
            for u in chain[i:]:
                Hi |= 1 << u
            Hi1 = Hi & ~(1 << v)
            p_v = sol.tgt_full[v] + min_over_supersets(Hi1) - min_over_supersets(Hi)
            assert abs((sol.tgt_full[v] - rfull[v]) - p_v) < 1e-13
            seen_outer += 1
    assert seen_outer > 20


def test_outer_residuals_hall_inequalities_and_sums():
    tight_seen = 0
    for tl, dl, n, topk in _outer_cases():
        sol = O.solve(tl, dl, n, topk, tol=1e-6, max_iter=10)
        k, js = sol.k, sol.jstar
        assert np.all(sol.p >= -1e-15) and np.all(sol.p <= sol.tgt_pos + 1e-15)
        dH = sol.drf_pos[:js].sum()
        assert abs(sol.p[js:].sum() - (1.0 - dH ** n)) < 1e-13           # equality at S = V \ H*
        assert abs(sol.residual_full().sum() - (1.0 - sol.alpha_star)) < 1e-13
        outer = list(range(js, k))
        # sum_S p <= phi(S) = 1 - (1 - drf(S))^n for every S of outer support tokens;
        # tight exactly on the unions of whole blocks counted from the lowest ratio
        for rsz in range(1, len(outer) + 1):
            for S in itertools.combinations(outer, rsz):
                S = list(S)
                lhs = sol.p[S].sum()
                phi = 1.0 - (1.0 - sol.drf_pos[S].sum()) ** n
                assert lhs <= phi + 1e-13
                blocks = set(sol.block[S].tolist())
                is_block_prefix = (set(S) == {j for j in outer if sol.block[j] in blocks}
                                   and blocks == set(range(max(blocks) + 1)))
                if is_block_prefix:
                    assert abs(lhs - phi) < 1e-13
                    tight_seen += 1
                else:
                    assert lhs < phi - 1e-9 or rsz == len(outer)
    assert tight_seen > 10


# ---------------------------------------------------------------- gradients (App. K; Thms 6.2)

@pytest.mark.parametrize("m,n", [(3, 2), (4, 3), (5, 2), (3, 4)])
def test_g1_and_g2_equal_tuple_enumeration_inner(m, n):
    rng = np.random.default_rng(m * 10 + n)
    d = rng.dirichlet(np.ones(m)) * 0.9
    w = np.exp(rng.normal(0, 2.0, m))
    ref = BF.inner_rowsums_enum(w, d, n)
    assert np.allclose(O.grad(O.ROUTE_G1, d, w, n), ref, rtol=0, atol=1e-13)
    assert np.allclose(O.grad(O.ROUTE_G2, d, w, n), ref, rtol=0, atol=1e-13)


@pytest.mark.parametrize("m,n,h", [(3, 2, 0.3), (4, 3, 0.1), (2, 4, 0.5), (4, 2, 0.0)])
def test_g1_and_g2_equal_tuple_enumeration_outer(m, n, h):
    rng = np.random.default_rng(m * 10 + n)
    d = rng.dirichlet(np.ones(m)) * (0.95 - h)
    w = np.exp(rng.normal(0, 1.5, m))
    ref = BF.outer_rowsums_enum(w, d, n, h)
    assert np.allclose(O.grad(O.ROUTE_G1, d, w, n, h=h, slack=False), ref, rtol=0, atol=1e-13)
    assert np.allclose(O.grad(O.ROUTE_G2, d, w, n, h=h, slack=False), ref, rtol=0, atol=1e-13)


@pytest.mark.parametrize("m,n", [(12, 8), (16, 5), (10, 16)])
def test_g2_equals_g1_on_larger_supports(m, n):
    rng = np.random.default_rng(m + n)
    d = rng.dirichlet(0.5 * np.ones(m))
    w = np.exp(rng.normal(0, 2.5, m))
    g1 = O.grad(O.ROUTE_G1, d, w, n)
    g2 = O.grad(O.ROUTE_G2, d, w, n)
    assert np.allclose(g1, g2, rtol=1e-9, atol=1e-12)
    g1o = O.grad(O.ROUTE_G1, d * 0.6, w, n, h=0.4, slack=False)
    g2o = O.grad(O.ROUTE_G2, d * 0.6, w, n, h=0.4, slack=False)
    assert np.allclose(g1o, g2o, rtol=1e-9, atol=1e-12)
    # total flow of an outer block is the mass of the tuples it serves
    assert abs(g2o.sum() - (1.0 - 0.4 ** n)) < 1e-12


# ---------------------------------------------------------------- the assembled coupling (Eqs. cases / approx-c)

def _coupling(sol, n):
    V = sol.V
    support = np.sort(sol.order)
    rfull = sol.residual_full()
    C = {}
    rowsum = np.zeros(V)
    accepted = 0.0
    for om in itertools.product(support.tolist(), repeat=n):
        pr = BF.draft_tuple_prob(sol.drf_full, om)
        nu, U, pi, rho = O.slice_(sol, list(om))
        assert nu == len(set(om))
        assert np.all(pi >= 0) and rho >= 0
        assert abs(pi.sum() + rho - 1.0) < 1e-12          # column sum = drf^n(omega)
        for t, x in zip(U, pi):
            rowsum[t] += pr * x
            accepted += pr * x
        if rho > 0:
            rowsum += pr * rho * rfull / rfull.sum()
            # resampled tokens never come from H* (Eq. res-zero)
            assert np.all(rfull[sol.order[: sol.jstar]] == 0)
        else:
            # outside (H*)^n the emitted token is always one of the drafts
            assert any(t not in set(sol.order[: sol.jstar].tolist()) for t in om) or sol.jstar == 0 or rho == 0
    return rowsum, accepted


def test_config1_coupling_has_exact_marginals():
    wl = W.config1(batch=12)
    tl = W.logits_to_f64(wl.q_logits); dl = W.logits_to_f64(wl.p_logits)
    multi_block = 0
    for b in range(12):
        sol = O.solve(tl[b], dl[b], wl.n, wl.topk, route=O.ROUTE_G2, tol=1e-13)
        assert sol.status == O.GRO_OK
        rowsum, acc = _coupling(sol, wl.n)
        assert np.abs(rowsum - sol.tgt_full).sum() < 1e-10      # emitted-token marginal is the target
        assert abs(acc - sol.alpha_star) < 1e-10                # and the acceptance is optimal
        multi_block += int(np.any(np.bincount(sol.block[sol.jstar:] + 1)[1:] > 1)) if sol.jstar < sol.k else 0
    assert multi_block > 0   # the outer softmax blocks were exercised


@pytest.mark.parametrize("V,n,topk,route", [(6, 3, 0, O.ROUTE_G1), (7, 3, 4, O.ROUTE_G2), (5, 4, 0, O.ROUTE_G2),
                                             (8, 2, 0, O.ROUTE_G1)])
def test_small_couplings_have_exact_marginals(V, n, topk, route):
    rng = np.random.default_rng(V * 100 + n)
    for _ in range(3):
        tl = 1.5 * rng.standard_normal(V); dl = tl + 1.0 * rng.standard_normal(V)
        sol = O.solve(tl, dl, n, topk, route=route, tol=1e-13)
        assert sol.status == O.GRO_OK
        rowsum, acc = _coupling(sol, n)
        assert np.abs(rowsum - sol.tgt_full).sum() < 1e-10
        assert abs(acc - sol.alpha_star) < 1e-10


def test_proportional_fitting_and_newton_reach_the_same_weights():
    """Two different iterations, one stopping test: the stationary point is unique."""
    rng = np.random.default_rng(78)
    for V, n, topk in [(12, 3, 0), (40, 4, 10), (16, 2, 0)]:
        tl = 1.5 * rng.standard_normal(V); dl = tl + 0.8 * rng.standard_normal(V)
        a = O.solve(tl, dl, n, topk, method=O.METHOD_IPF, tol=1e-12, max_iter=400000)
        b = O.solve(tl, dl, n, topk, method=O.METHOD_NEWTON, tol=1e-12)
        assert a.status == O.GRO_OK and b.status == O.GRO_OK
        assert np.allclose(a.w, b.w, rtol=1e-7)


def test_both_routes_reach_the_same_weights():
    rng = np.random.default_rng(77)
    tl = 1.5 * rng.standard_normal(12); dl = tl + 1.0 * rng.standard_normal(12)
    a = O.solve(tl, dl, 3, 0, route=O.ROUTE_G1, tol=1e-13)
    b = O.solve(tl, dl, 3, 0, route=O.ROUTE_G2, tol=1e-13)
    assert a.jstar == b.jstar and np.array_equal(a.block, b.block)
    assert np.allclose(a.w, b.w, rtol=1e-8)


# ---------------------------------------------------------------- the draw (App. A steps 3-4)

def test_draw_segments_and_boundaries():
    U = np.array([5, 2, 9], dtype=np.int32)
    pi = np.array([0.25, 0.0, 0.5])
    rho = 0.25
    r = np.zeros(12); r[[0, 3, 7, 11]] = [0.1, 0.2, 0.3, 0.4]
    eps = 1e-12
    assert O.draw(U, pi, rho, r, 0.0, 0.5) == (5, 1)
    assert O.draw(U, pi, rho, r, 0.25 - eps, 0.5) == (5, 1)
    assert O.draw(U, pi, rho, r, 0.25, 0.5) == (9, 1)          # zero-width segment of token 2 is skipped
    assert O.draw(U, pi, rho, r, 0.75 - eps, 0.5) == (9, 1)
    assert O.draw(U, pi, rho, r, 0.75, 0.0) == (0, 0)
    assert O.draw(U, pi, rho, r, 0.9, 0.1 - eps) == (0, 0)
    assert O.draw(U, pi, rho, r, 0.9, 0.1 + eps) == (3, 0)
    assert O.draw(U, pi, rho, r, 0.9, 0.3 + eps) == (7, 0)
    assert O.draw(U, pi, rho, r, 0.9, 0.999999) == (11, 0)


def test_draw_integrates_to_the_slice_and_target_marginal():
    wl = W.config1(batch=1)
    tl = W.logits_to_f64(wl.q_logits)[0]; dl = W.logits_to_f64(wl.p_logits)[0]
    sol = O.solve(tl, dl, 2, 0, tol=1e-13)
    rfull = sol.residual_full()
    rng = np.random.default_rng(0)
    N = 120000
    cdf = np.cumsum(sol.drf_full)
    hist = np.zeros(sol.V); acc = 0
    cache = {}
    draws = np.searchsorted(cdf, rng.random((N, 2)) * cdf[-1], side="right").clip(max=sol.V - 1)
    us = rng.random((N, 2))
    for om, (u0, u1) in zip(draws, us):
        key = (int(om[0]), int(om[1]))
        if key not in cache:
            cache[key] = O.slice_(sol, om)
        nu, U, pi, rho = cache[key]
        tok, a = O.draw(U, pi, rho, rfull, u0, u1)
        hist[tok] += 1; acc += a
        assert (tok in key) == bool(a)
    sigma = np.sqrt(sol.tgt_full * (1 - sol.tgt_full) / N)
    assert np.all(np.abs(hist / N - sol.tgt_full) < 5 * sigma + 1e-4)
    assert abs(acc / N - sol.alpha_star) < 5 * np.sqrt(0.25 / N)


def test_batch_driver_matches_single_calls():
    wl = W.config1(batch=6)
    tl = W.logits_to_f64(wl.q_logits); dl = W.logits_to_f64(wl.p_logits)
    res = O.solve_verify_batch(tl, dl, wl.n, wl.topk, 1.0, 1.0, wl.draft_tokens.numpy(), wl.uniforms.numpy())
    for b in range(6):
        sol = O.solve(tl[b], dl[b], wl.n, wl.topk)
        assert abs(res.alpha_star[b] - sol.alpha_star) < 1e-15
        nu, U, pi, rho = O.slice_(sol, wl.draft_tokens[b].numpy())
        assert np.allclose(res.pi[b, :nu], pi) and abs(res.rho[b] - rho) < 1e-15
        tok, a = O.draw(U, pi, rho, sol.residual_full(), float(wl.uniforms[b, 0]), float(wl.uniforms[b, 1]))
        assert (res.token[b], res.accepted[b]) == (tok, a)


def test_draft_token_outside_support_is_an_error():
    rng = np.random.default_rng(1)
    tl, dl = _rand_logits(rng, 10)
    sol = O.solve(tl, dl, 2, 3)
    outside = [i for i in range(10) if i not in sol.order.tolist()][0]
    nu, *_ = O.slice_(sol, [int(sol.order[0]), outside])
    assert nu == O.GRO_DRAFT_OUT_OF_SUPPORT


def test_golden_config1_values_have_not_drifted():
    """tests/golden/config1_oracle.txt was written by tests/golden/make_golden.py from the oracle alone."""
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "config1_oracle.txt")
    rows = [ln.split() for ln in open(path) if not ln.startswith("#")]
    wl = W.config1(batch=8)
    tl = W.logits_to_f64(wl.q_logits); dl = W.logits_to_f64(wl.p_logits)
    for b, a, js, nb in rows:
        sol = O.solve(tl[int(b)], dl[int(b)], wl.n, wl.topk, tol=1e-12)
        assert abs(sol.alpha_star - float(a)) < 1e-13 and sol.jstar == int(js) and sol.nblocks == int(nb)


def test_alpha_star_only_agrees_with_the_full_solve_and_with_enumeration():
    rng = np.random.default_rng(314)
    for V, n, topk in [(10, 3, 0), (12, 2, 5), (9, 8, 0)]:
        tl, dl = _rand_logits(rng, V)
        a, js = O.alpha_star_only(tl, dl, n, topk)
        sol = O.solve(tl, dl, n, topk, tol=1e-6, max_iter=5)
        assert a == sol.alpha_star and js == sol.jstar
        tgt, drf, _, _ = O.distributions(tl, dl, topk, 1.0, 1.0)
        assert abs(a - (1.0 + BF.all_subset_psi(tgt, drf, n).min())) < 1e-13


# ---------------------------------------------------------------- truncated variant (Sec. 6.2-6.3, Algorithm 1)

def test_truncation_sets_are_minimal_and_meet_their_bounds():
    rng = np.random.default_rng(631)
    for V, n, tau in [(9, 2, 0.05), (10, 3, 0.01), (8, 4, 0.2), (10, 2, 1e-4)]:
        for _ in range(4):
            tl = 1.5 * rng.standard_normal(V); dl = tl + 1.2 * rng.standard_normal(V)
            sol = O.solve(tl, dl, n, 0, tol=1e-6, max_iter=20)
            k, js = sol.k, sol.jstar
            in_T, gam, eps = O.truncation_sets(sol.order, sol.drf_pos, js, n, tau)
            d = sol.drf_pos
            D = d[:js].sum()
            Tin = [j for j in range(js) if in_T[j]]; Tout = [j for j in range(js, k) if in_T[j]]
            assert abs(gam - (D ** n - d[Tin].sum() ** n)) < 1e-14 and gam <= tau
            assert abs(eps - (1.0 - (D + d[Tout].sum()) ** n)) < 1e-14 and eps <= tau
            # no smaller subset meets the bound (all subsets of one size less)
            if Tin:
                best = max(d[list(S)].sum() for S in itertools.combinations(range(js), len(Tin) - 1)) if len(Tin) > 1 else 0.0
                assert D ** n - best ** n > tau
            if Tout:
                best = max(d[list(S)].sum() for S in itertools.combinations(range(js, k), len(Tout) - 1)) if len(Tout) > 1 else 0.0
                assert 1.0 - (D + best) ** n > tau
    # tau = 0 keeps every support token
    in_T, gam, eps = O.truncation_sets(sol.order, sol.drf_pos, sol.jstar, n, 0.0)
    assert in_T.all() and gam == 0.0 and eps == 0.0


@pytest.mark.parametrize("V,n,topk", [(7, 2, 0), (8, 3, 0), (8, 2, 5), (6, 4, 0)])
def test_truncated_rule_keeps_the_papers_guarantees(V, n, topk):
    """The coupling assembled from the truncated solves (all tuples enumerated): within 15 tau of the target in L1,
    acceptance within 10 tau of the optimum, column sums exact (Lemma "Approximation Guarantee", Sec. 6.3)."""
    rng = np.random.default_rng(V * 1000 + n * 10 + topk)
    used_truncation = 0
    for tau in (0.1, 0.02, 1e-3):
        for _ in range(3):
            tl = 1.5 * rng.standard_normal(V); dl = tl + 1.0 * rng.standard_normal(V)
            sol = O.solve(tl, dl, n, topk, tau=tau)
            used_truncation += int(np.any(sol.w[: sol.k] == 0.0))
            rowsum, acc = _coupling(sol, n)
            assert np.abs(rowsum - sol.tgt_full).sum() <= 15 * tau
            assert abs(acc - sol.alpha_star) <= 10 * tau
            # the marginals computed without enumeration agree with the enumerated ones
            l1, acc2, flow = O.rule_deviation(sol)
            assert abs(l1 - np.abs(rowsum - sol.tgt_full).sum()) < 1e-11
            assert abs(acc2 - acc) < 1e-11
    assert used_truncation > 0


def test_truncated_rule_tends_to_the_exact_one():
    rng = np.random.default_rng(99)
    tl = 1.5 * rng.standard_normal(12); dl = tl + 0.9 * rng.standard_normal(12)
    exact = O.solve(tl, dl, 3, 0, tol=1e-13)
    tiny = O.solve(tl, dl, 3, 0, tau=1e-14)
    assert np.all(tiny.w[: tiny.k] > 0)
    assert np.allclose(tiny.w, exact.w, rtol=1e-6)
    devs = [O.rule_deviation(O.solve(tl, dl, 3, 0, tau=t))[0] for t in (0.1, 1e-2, 1e-3, 1e-5)]
    assert devs[-1] < 1e-4 and devs[-1] <= devs[0] + 1e-12


def test_rule_marginals_for_arbitrary_weights_match_enumeration():
    """gro_rule_deviation against the enumerated coupling for weights that solve nothing, zeros included
    (whole blocks of zeros share their tuples equally)."""
    rng = np.random.default_rng(5150)
    seen_zero_block = 0
    for V, n, topk in [(7, 3, 0), (8, 2, 0), (7, 2, 5)]:
        for _ in range(4):
            tl = 1.5 * rng.standard_normal(V); dl = tl + 1.3 * rng.standard_normal(V)
            sol = O.solve(tl, dl, n, topk, tol=1e-6, max_iter=30)
            w = np.exp(rng.normal(0, 1.5, sol.k))
            w[rng.random(sol.k) < 0.4] = 0.0
            for b in range(sol.nblocks):
                if rng.random() < 0.3:
                    w[sol.block[: sol.k] == b] = 0.0
                    seen_zero_block += 1
            sol2 = O.Solution(**{**sol.__dict__, "w": w})
            rowsum, acc = _coupling(sol2, n)
            l1, acc2, flow = O.rule_deviation(sol, w)
            assert abs(acc2 - acc) < 1e-11
            assert abs(l1 - np.abs(rowsum - sol.tgt_full).sum()) < 1e-11
    assert seen_zero_block > 0


def test_certificate_and_draw_sweep_helpers():
    """The batch helpers used by the GPU tests: the certificate vanishes at the oracle's own weights and does not at
    perturbed ones; the sweep's first draw is the batch driver's draw."""
    wl = W.config1(batch=6)
    tl = W.logits_to_f64(wl.q_logits); dl = W.logits_to_f64(wl.p_logits)
    tk = wl.draft_tokens.numpy(); un = wl.uniforms.numpy()
    res = O.solve_verify_batch(tl, dl, wl.n, wl.topk, 1.0, 1.0, tk, un)
    cert = O.certify_batch(tl, dl, wl.n, wl.topk, 1.0, 1.0, res.w, lse=None)
    assert cert.gnorm.max() < 1e-11 and np.array_equal(cert.order, res.order) and np.array_equal(cert.block, res.block)
    bad = O.certify_batch(tl, dl, wl.n, wl.topk, 1.0, 1.0, res.w * (1.0 + 0.01 * (np.arange(res.w.shape[1]) % 3)))
    solved = [b for b in range(6) if res.jstar[b] >= 2 or np.any(np.bincount(res.block[b][res.block[b] >= 0]) >= 2)]
    assert all(bad.gnorm[b] > 1e-6 for b in solved) and len(solved) >= 3
    # a log-sum-exp given from outside: off by delta, the certificate against the shifted target sees ~delta
    shifted = O.certify_batch(tl, dl, wl.n, wl.topk, 1.0, 1.0, res.w, lse=cert.lse_target + 1e-6)
    assert np.all(shifted.gnorm_lse[solved] > 1e-8) and shifted.gnorm.max() < 1e-11
    tok, acc, margin = O.draw_sweep_batch(tl, dl, wl.n, wl.topk, 1.0, 1.0, res, tk, un[:, None, :])
    assert np.array_equal(tok[:, 0], res.token) and np.array_equal(acc[:, 0], res.accepted) and np.all(margin >= 0)
