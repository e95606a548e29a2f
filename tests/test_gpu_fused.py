"""gr_solve_verify (one call: the solve kernel finishes every instance with its draw, and solves only the
system the drafted tuple selects) against gr_solve + gr_verify, whose parity with the oracle the other
GPU tests establish, and against the oracle's emitted tokens directly."""
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


def _both(wl, opt=None):
    solved = G.solve(wl.q_logits, wl.p_logits, wl.n, wl.topk, wl.temp_target, wl.temp_draft, opt)
    ver = G.verify(solved, wl.draft_tokens, wl.uniforms)
    sv, vf = G.solve_verify(wl.q_logits, wl.p_logits, wl.draft_tokens, wl.uniforms, wl.topk, wl.temp_target,
                            wl.temp_draft, opt)
    torch.cuda.synchronize()
    return solved, ver, sv, vf


def _same_draws(ver, vf):
    assert torch.equal(ver.token.cpu(), vf.token.cpu())
    assert torch.equal(ver.accepted.cpu(), vf.accepted.cpu())
    assert torch.equal(ver.status.cpu(), vf.status.cpu())


@pytest.mark.parametrize("make", [
    lambda: W.config1(device="cuda"),
    lambda: W.config2(device="cuda"),
    lambda: W.config3(batch=96, device="cuda"),
    lambda: W.config4(8, 20, 1.0, batch=128, device="cuda"),
    lambda: W.config4(16, 5, 2.0, batch=128, device="cuda"),
    lambda: W.config5(batch=24, device="cuda"),
])
def test_fused_call_emits_the_tokens_of_the_two_call_path(make):
    wl = make()
    solved, ver, sv, vf = _both(wl)
    _same_draws(ver, vf)
    assert torch.equal(solved.alpha_star.cpu(), sv.alpha_star.cpu())


def test_fused_call_matches_the_oracle_tokens_on_config1():
    """Config 1 has outer blocks in most instances, so the selective solve is exercised: tokens against the oracle."""
    wl = W.config1(device="cuda")
    sv, vf = G.solve_verify(wl.q_logits, wl.p_logits, wl.draft_tokens, wl.uniforms, wl.topk, wl.temp_target,
                            wl.temp_draft)
    torch.cuda.synchronize()
    tl = W.logits_to_f64(wl.q_logits); dl = W.logits_to_f64(wl.p_logits)
    toks = wl.draft_tokens.cpu().numpy(); uni = wl.uniforms.cpu().numpy()
    res = O.solve_verify_batch(tl, dl, wl.n, wl.topk, wl.temp_target, wl.temp_draft, toks, uni, tol=1e-11)
    g_tok = vf.token.cpu().numpy(); g_acc = vf.accepted.cpu().numpy()
    bad = 0
    for b in range(wl.batch):
        if g_tok[b] != res.token[b] or int(g_acc[b]) != int(res.accepted[b]):
            # excused only when a uniform sits within 1e-6 of a boundary of the oracle's CDFs
            sol = O.solve(tl[b], dl[b], wl.n, wl.topk, wl.temp_target, wl.temp_draft, tol=1e-11)
            nu, U, pi, rho = O.slice_(sol, toks[b])
            close = np.min(np.abs(np.cumsum(pi) - uni[b, 0])) < 1e-6
            if not close and rho > 0:
                rf = sol.residual_full(); cdf = np.cumsum(rf) / rf.sum()
                close = np.min(np.abs(cdf - uni[b, 1])) < 1e-6
            bad += 0 if close else 1
    assert bad == 0
    assert np.max(np.abs(sv.alpha_star.cpu().numpy() - res.alpha_star)) <= 1e-6


def test_partial_rules_are_marked_and_refused_by_gr_verify():
    wl = W.config1(device="cuda")
    solved, ver, sv, vf = _both(wl)
    rule = G.read_rule(sv)
    full = G.read_rule(solved)
    torch.cuda.synchronize()
    partial = (rule.status == G.GR_PARTIAL_RULE).numpy()
    # an instance is partial exactly when a system with unknowns other than the selected one exists
    toks = wl.draft_tokens.cpu().numpy()
    expect = np.zeros(wl.batch, dtype=bool)
    for b in range(wl.batch):
        k = int(full.k[b]); js = int(full.jstar[b])
        ids = full.ids[b, :k].numpy().tolist(); blk = full.block[b, :k].numpy()
        systems = set(["inner"] if js > 0 else [])
        systems |= {int(v) for v in set(blk[js:].tolist()) if (blk == v).sum() >= 2}
        maxpos = max(ids.index(int(t)) for t in toks[b])
        sel = "inner" if maxpos < js else int(blk[maxpos])
        expect[b] = len(systems - {sel}) > 0
    assert partial.any() and np.array_equal(partial, expect)
    # the system that was solved carries the weights of the full solve
    again = G.verify(sv, wl.draft_tokens, wl.uniforms)
    torch.cuda.synchronize()
    st = again.status.cpu().numpy(); tk = again.token.cpu().numpy()
    assert np.all(st[partial] == G.GR_PARTIAL_RULE) and np.all(tk[partial] == -1)
    assert np.array_equal(tk[~partial], ver.token.cpu().numpy()[~partial])


def test_fused_call_on_the_general_kernel_and_error_statuses():
    wl = W.config2(batch=4, device="cuda", V=5000)
    q = wl.q_logits.clone(); p = wl.p_logits.clone()
    q[1, 123] = float("nan")
    toks = wl.draft_tokens.clone()
    sup = torch.topk(wl.p_logits[3], 8).indices
    toks[3, 1] = [i for i in range(100) if i not in sup.tolist()][0]
    for opt in (None, G.Options(force_robust=1)):
        solved = G.solve(q, p, wl.n, wl.topk, 1.0, 1.0, opt)
        ver = G.verify(solved, toks, wl.uniforms)
        sv, vf = G.solve_verify(q, p, toks, wl.uniforms, wl.topk, 1.0, 1.0, opt)
        torch.cuda.synchronize()
        _same_draws(ver, vf)
        vs = vf.status.cpu().tolist(); tk = vf.token.cpu().tolist()
        assert vs[0] == G.GR_OK and tk[0] >= 0
        assert vs[1] == G.GR_BAD_LOGITS and tk[1] == -1
        assert vs[3] == G.GR_DRAFT_OUT_OF_SUPPORT and tk[3] == -1


def test_fused_call_without_a_rule_samples_the_target():
    wl = W.config4(4, 0, 1.0, batch=6, device="cuda", V=5000, seed=99)
    solved, ver, sv, vf = _both(wl)
    _same_draws(ver, vf)
    assert vf.status.cpu().tolist() == [G.GR_SUPPORT_TOO_LARGE] * 6
    assert torch.equal(solved.alpha_star.cpu(), sv.alpha_star.cpu())


def test_fused_call_rejects_missing_pointers():
    wl = W.config2(batch=2, device="cuda", V=5000)
    sv = G.solve(wl.q_logits, wl.p_logits, wl.n, wl.topk)
    rc = G.gr_solve_verify(wl.q_logits.data_ptr(), wl.p_logits.data_ptr(), G.GR_F32, wl.V, wl.n, wl.topk, 1.0, 1.0, 2,
                           None, 0, wl.uniforms.data_ptr(), sv.params.data_ptr(), sv.workspace.data_ptr(),
                           sv.alpha_star.data_ptr(), 0, 0, sv.status.data_ptr(), 0)
    assert rc == -2
