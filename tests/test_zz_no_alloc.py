"""gr_solve_static: the variant of gr_solve for callers that cannot allocate device memory
(a serving loop whose pool owns all free memory, a host that may not call cudaMalloc once running).

It keeps its scratch in a fixed array inside the library, so it takes no workspace.  The test
calls it through the C interface twice in a row, on different inputs, and checks that the rule,
the optimal acceptance and the emitted tokens equal those of gr_solve with a caller-owned
workspace (same kernels, so equality is exact; the acceptance is also held to the 1e-6 used
elsewhere).  The second call sees the first call's leftovers in the shared scratch.
This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

import paper_2511_15898_b200 as G
from paper_2511_15898_b200 import workloads as W
from paper_2511_15898_b200.build import build_library

pytestmark = pytest.mark.gpu


def _static_solve(wl):
    """Outputs are ordinary caller-owned tensors; only the scratch comes from the library."""
    B = wl.batch
    dev = wl.q_logits.device
    params = torch.empty(G.gr_params_bytes(wl.V, wl.n, wl.topk, B), dtype=torch.uint8, device=dev)
    alpha = torch.empty(B, dtype=torch.float32, device=dev)
    status = torch.empty(B, dtype=torch.int32, device=dev)
    dtype = G.GR_BF16 if wl.q_logits.dtype == torch.bfloat16 else G.GR_F32
    rc = G.gr_solve_static(wl.q_logits.data_ptr(), wl.p_logits.data_ptr(), dtype, wl.V, wl.n, wl.topk,
                           wl.temp_target, wl.temp_draft, B, None, params.data_ptr(), alpha.data_ptr(),
                           status.data_ptr(), int(torch.cuda.current_stream().cuda_stream))
    assert rc == 0, G.gr_strerror(rc)
    return G.binding.Solved(wl.V, wl.n, wl.topk, B, params, torch.empty(0, dtype=torch.uint8, device=dev), alpha,
                            status, wl.q_logits)


def _same(wl):
    ref = G.solve(wl.q_logits, wl.p_logits, wl.n, wl.topk, wl.temp_target, wl.temp_draft)
    ref_v = G.verify(ref, wl.draft_tokens, wl.uniforms)
    ref_rule = G.read_rule(ref)
    got = _static_solve(wl)
    got_v = G.verify(got, wl.draft_tokens, wl.uniforms)
    got_rule = G.read_rule(got)
    torch.cuda.synchronize()
    assert torch.equal(got.status, ref.status)
    assert float((got.alpha_star - ref.alpha_star).abs().max()) <= 1e-6
    assert torch.equal(got_rule.ids, ref_rule.ids) and torch.equal(got_rule.block, ref_rule.block)
    assert np.allclose(got_rule.w.numpy(), ref_rule.w.numpy(), rtol=1e-9, atol=0)
    assert torch.equal(got_v.token, ref_v.token) and torch.equal(got_v.accepted, ref_v.accepted)


def test_static_scratch_matches_caller_workspace_on_two_calls_in_a_row():
    build_library()
    _same(W.config2(batch=48, device="cuda", V=12000))
    # different shape and content: whatever the first call left in the shared scratch must not matter
    _same(W.config3(batch=20, device="cuda", V=40000, n=4, topk=24))


def test_static_call_leaves_free_device_memory_unchanged():
    """What the entry point is for: after its first call on the device (which looks up the built-in array's
    address) a call allocates nothing.  Free device memory as the driver reports it is the same before and after
    a call whose outputs were allocated beforehand."""
    build_library()
    wl = W.config2(batch=32, device="cuda", V=9000)
    _static_solve(wl)                      # first call on this device: set-up
    B = wl.batch
    dev = wl.q_logits.device
    params = torch.empty(G.gr_params_bytes(wl.V, wl.n, wl.topk, B), dtype=torch.uint8, device=dev)
    alpha = torch.empty(B, dtype=torch.float32, device=dev)
    status = torch.empty(B, dtype=torch.int32, device=dev)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        rc = G.gr_solve_static(wl.q_logits.data_ptr(), wl.p_logits.data_ptr(), G.GR_F32, wl.V, wl.n, wl.topk,
                               wl.temp_target, wl.temp_draft, B, None, params.data_ptr(), alpha.data_ptr(),
                               status.data_ptr(), int(torch.cuda.current_stream().cuda_stream))
        assert rc == 0
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, (free0, free1)
    assert status.cpu().tolist() == [G.GR_OK] * B


def test_static_scratch_rejects_what_it_cannot_hold():
    build_library()
    A = 1 << 20
    rc = G.gr_solve_static(A, A, G.GR_F32, 1000, 2, 8, 1.0, 1.0, G.GR_STATIC_MAX_BATCH + 1, None, A, A, A, 0)
    assert rc == -5 and "capacity" in G.gr_strerror(rc)
    assert G.gr_solve_static(A, A, G.GR_F32, 1000, 2, 8, 1.0, 1.0, 0, None, A, A, A, 0) == 0
    # an untruncated draft on a vocabulary beyond the solve capacity needs a per-row sort buffer the scratch lacks
    assert G.gr_solve_static(A, A, G.GR_F32, 100000, 2, 0, 1.0, 1.0, 2, None, A, A, A, 0) == -5
