"""The truncated variant on the GPU (gr_options.tau; Sec. 6.2 tunable errors, Sec. 6.3, Algorithm 1).

Any point with gradient norm <= 5 tau is an admissible answer, so the weights are not compared one by one with
the oracle's.  What is compared: the truncation sets (the zero pattern of the weights), the paper's guarantees
for the GPU's rule -- L1 distance of the emitted-token marginal from the target <= 15 tau, acceptance within
10 tau of the optimum, both evaluated by the oracle for the GPU's weights -- the emitted tokens against the
oracle's draw from that same rule, and tau -> 0 against the exact rule.
"""
import dataclasses

import numpy as np
import pytest
import torch

import paper_2511_15898_b200 as G
from paper_2511_15898_b200 import workloads as W
from paper_2511_15898_b200.build import build_library
from oracle import gr_oracle as O
from tests import parity as P

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build_library()
    G.load_library()


def _check_tau(wl, tau, draws=8, force_robust=0):
    opt = G.Options(tau=tau, force_robust=force_robust)
    solved = G.solve(wl.q_logits, wl.p_logits, wl.n, wl.topk, wl.temp_target, wl.temp_draft, opt)
    rule = G.read_rule(solved)
    torch.cuda.synchronize()
    assert solved.status.cpu().tolist() == [G.GR_OK] * wl.batch
    tl = W.logits_to_f64(wl.q_logits); dl = W.logits_to_f64(wl.p_logits)
    toks = wl.draft_tokens.cpu().numpy(); uni = wl.uniforms.cpu().numpy()
    res = O.solve_verify_batch(tl, dl, wl.n, wl.topk, wl.temp_target, wl.temp_draft, toks, uni, tau=tau)
    g_w = rule.w.numpy()
    l1_max = 0.0; acc_dev = 0.0; truncated = 0; near = 0
    for b in range(wl.batch):
        k = int(res.k[b]); js = int(res.jstar[b])
        if P.near_tie(res.psi[b], k, js, wl.V, 1e-6):
            near += 1
            continue
        assert int(rule.jstar[b]) == js and np.array_equal(rule.ids[b, :k].numpy(), res.order[b, :k])
        assert np.array_equal(rule.block[b, :k].numpy(), res.block[b, :k])
        # the same truncation sets: zero weights in the same places
        assert np.array_equal(g_w[b, :k] == 0.0, res.w[b, :k] == 0.0), (b, g_w[b, :k], res.w[b, :k])
        truncated += int(np.any(g_w[b, :k] == 0.0))
        sol = O.solve(tl[b], dl[b], wl.n, wl.topk, wl.temp_target, wl.temp_draft, tau=tau)
        l1, acc, _ = O.rule_deviation(sol, g_w[b, :k])
        l1_max = max(l1_max, l1); acc_dev = max(acc_dev, abs(acc - sol.alpha_star))
    print(f"tau={tau:g}: instances with a truncated system {truncated}/{wl.batch}, L1 to target max {l1_max:.3e} "
          f"(bound {15 * tau:.3e}), acceptance deviation max {acc_dev:.3e} (bound {10 * tau:.3e}), near ties {near}")
    assert l1_max <= 15 * tau and acc_dev <= 10 * tau
    assert near <= max(1, wl.batch // 50)
    # the draw from the GPU's own rule: the oracle draws from the same weights
    res_g = dataclasses.replace(res, w=g_w[:, : res.w.shape[1]].copy())
    U = np.empty((wl.batch, draws, 2), dtype=np.float32)
    U[:, 0, :] = uni
    U[:, 1:, :] = P._sweep_uniforms(wl.batch, draws - 1, res.rho, seed=int(tau * 1e6) + wl.V)
    o_tok, o_acc, margin = O.draw_sweep_batch(tl, dl, wl.n, wl.topk, wl.temp_target, wl.temp_draft, res_g, toks, U)
    bad = 0
    for q in range(draws):
        uq = torch.from_numpy(np.ascontiguousarray(U[:, q, :])).to(wl.q_logits.device)
        ver = G.verify(solved, wl.draft_tokens, uq)
        torch.cuda.synchronize()
        gt = ver.token.cpu().numpy(); ga = ver.accepted.cpu().numpy()
        diff = (gt != o_tok[:, q]) | (ga != o_acc[:, q])
        bad += int(np.sum(diff & (margin[:, q] >= 1e-6)))
    assert bad == 0
    return truncated


@pytest.mark.parametrize("tau", [5e-2, 1e-2, 1e-3])
def test_truncated_headline_shape(tau):
    """With 8 drafts a token can only be left out when 1 - (1 - its mass)^8 <= tau: at the headline shape (smallest of
    the 50 draft masses ~4e-3) the sets only shrink from tau ~ 0.03 on; below that the dial is the looser stop alone."""
    tr = _check_tau(W.config3(batch=48, device="cuda", seed=3011), tau)
    assert tr > 0 or tau < 3e-2


def test_truncated_tiny_full_support_with_outer_blocks():
    _check_tau(W.config1(device="cuda"), 2e-2)
    _check_tau(W.config1(device="cuda"), 1e-3)


def test_truncated_config2_and_config4_cell():
    _check_tau(W.config2(batch=48, device="cuda"), 1e-2)
    _check_tau(W.config4(8, 20, 1.0, batch=32, device="cuda"), 1e-2)


def test_truncated_robust_kernel_and_32_drafts():
    _check_tau(W.config4(32, 20, 1.0, batch=16, device="cuda"), 1e-2)
    _check_tau(W.config3(batch=12, device="cuda", seed=3012), 1e-2, force_robust=1)


def test_truncated_wide_support():
    tr = _check_tau(W.config5(batch=16, device="cuda", rows_per_pass=16), 5e-2)
    assert tr > 0


def test_vanishing_tau_reproduces_the_exact_rule():
    wl = W.config3(batch=24, device="cuda", seed=3013)
    exact = G.read_rule(G.solve(wl.q_logits, wl.p_logits, wl.n, wl.topk, wl.temp_target, wl.temp_draft))
    tiny = G.read_rule(G.solve(wl.q_logits, wl.p_logits, wl.n, wl.topk, wl.temp_target, wl.temp_draft,
                               G.Options(tau=1e-13)))
    torch.cuda.synchronize()
    assert bool((tiny.w[exact.w > 0] > 0).all())
    assert float(((tiny.w - exact.w).abs() / exact.w.clamp_min(1e-300))[exact.w > 0].max()) < 1e-5


def test_tau_out_of_range_is_rejected():
    wl = W.config2(batch=2, device="cuda", V=4000)
    for bad in (-1e-3, 1.5, float("nan")):
        with pytest.raises(G.GrError):
            G.solve(wl.q_logits, wl.p_logits, wl.n, wl.topk, opt=G.Options(tau=bad))
