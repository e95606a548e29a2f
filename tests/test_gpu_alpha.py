"""gr_alpha_star (optimal acceptance for several draft counts from one pass over the logits) against the
oracle's subset selection and against gr_solve."""
import numpy as np
import pytest
import torch

import paper_2511_15898_b200 as G
from paper_2511_15898_b200 import workloads as W
from paper_2511_15898_b200.build import build_library
from oracle import gr_oracle as O

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build_library()
    G.load_library()


@pytest.mark.parametrize("make", [
    lambda: W.config1(device="cuda"),
    lambda: W.config2(batch=48, device="cuda"),
    lambda: W.config3(batch=24, device="cuda"),
    lambda: W.config4(8, 20, 2.0, batch=32, device="cuda"),
    lambda: W.config5(batch=12, device="cuda"),
])
def test_alpha_star_for_several_draft_counts_matches_the_oracle(make):
    wl = make()
    ns = [1, 2, 3, 4, 8, 16, 32]
    out, st = G.alpha_star(wl.q_logits, wl.p_logits, ns, wl.topk, wl.temp_target, wl.temp_draft)
    torch.cuda.synchronize()
    assert st.cpu().tolist() == [G.GR_OK] * wl.batch
    got = out.cpu().numpy().astype(np.float64)
    tl = W.logits_to_f64(wl.q_logits); dl = W.logits_to_f64(wl.p_logits)
    for b in range(wl.batch):
        for e, n in enumerate(ns):
            a, _ = O.alpha_star_only(tl[b], dl[b], n, wl.topk, wl.temp_target, wl.temp_draft)
            assert abs(got[b, e] - a) <= 1e-6, (b, n, got[b, e], a)
    # the acceptance grows with the number of drafts (more tuples can only help)
    assert np.all(np.diff(got, axis=1) >= -1e-6)
    # and the column of the workload's own n is what gr_solve reports
    if wl.n in ns:
        solved = G.solve(wl.q_logits, wl.p_logits, wl.n, wl.topk, wl.temp_target, wl.temp_draft)
        torch.cuda.synchronize()
        assert np.max(np.abs(solved.alpha_star.cpu().numpy() - got[:, ns.index(wl.n)])) <= 1e-6


def test_alpha_star_argument_checks_and_bad_rows():
    wl = W.config2(batch=3, device="cuda", V=5000)
    q = wl.q_logits.clone()
    q[1, 17] = float("nan")
    out, st = G.alpha_star(q, wl.p_logits, [2, 4], wl.topk)
    torch.cuda.synchronize()
    assert st.cpu().tolist() == [G.GR_OK, G.GR_BAD_LOGITS, G.GR_OK]
    assert torch.isnan(out[1]).all() and not torch.isnan(out[0]).any()
    with pytest.raises(G.GrError):
        G.alpha_star(q, wl.p_logits, [], wl.topk)
    with pytest.raises(G.GrError):
        G.alpha_star(q, wl.p_logits, [0], wl.topk)
    with pytest.raises(G.GrError):
        G.alpha_star(q, wl.p_logits, list(range(1, 10)), wl.topk)
    with pytest.raises(G.GrError):                       # a truncated support beyond the capacity
        G.alpha_star(q, wl.p_logits, [2], 500)


@pytest.mark.parametrize("V,sigma", [(50257, 1.0), (7001, 0.25), (129, 2.0)])
def test_alpha_star_of_an_untruncated_draft_on_a_large_vocabulary(V, sigma):
    """Whole-vocabulary draft, V beyond the rule's capacity: the minimum of psi is searched per draft count without a
    params block; the values must equal the oracle's subset selection and what gr_solve reports for the same n,
    and a row with a NaN is reported as such."""
    wl = W.config4(8, 0, sigma, batch=6, device="cuda", V=V, seed=900 + V % 97)
    ns = [1, 2, 4, 8, 32]
    q = wl.q_logits.clone()
    q[4, 5] = float("nan")
    out, st = G.alpha_star(q, wl.p_logits, ns, 0, wl.temp_target, wl.temp_draft)
    torch.cuda.synchronize()
    assert st.cpu().tolist() == [G.GR_OK] * 4 + [G.GR_BAD_LOGITS, G.GR_OK]
    assert torch.isnan(out[4]).all()
    got = out.cpu().numpy().astype(np.float64)
    tl = W.logits_to_f64(wl.q_logits); dl = W.logits_to_f64(wl.p_logits)
    for b in (0, 1, 2, 3, 5):
        for e, n in enumerate(ns):
            a, _ = O.alpha_star_only(tl[b], dl[b], n, 0, wl.temp_target, wl.temp_draft)
            assert abs(got[b, e] - a) <= 1e-6, (b, n, got[b, e], a)
        assert np.all(np.diff(got[b]) >= -1e-6)
    solved = G.solve(wl.q_logits, wl.p_logits, 8, 0, wl.temp_target, wl.temp_draft)
    torch.cuda.synchronize()
    ref = solved.alpha_star.cpu().numpy()
    assert np.max(np.abs(ref[[0, 1, 2, 3, 5]] - got[[0, 1, 2, 3, 5], ns.index(8)])) <= 1e-6
