"""The synthetic workloads have the stated shapes, dtypes and structure, and are reproducible."""
import numpy as np
import torch

from paper_2511_15898_b200 import workloads as W


def test_config1_shape_and_seed():
    a = W.config1(); b = W.config1()
    assert a.q_logits.shape == (64, 16) and a.n == 2 and a.topk == 0
    assert torch.equal(a.q_logits, b.q_logits) and torch.equal(a.draft_tokens, b.draft_tokens)
    assert a.uniforms.shape == (64, 2) and float(a.uniforms.min()) >= 0 and float(a.uniforms.max()) < 1


def test_topk_draft_tokens_lie_in_the_support():
    wl = W.config2(batch=8, V=4000)
    top = torch.topk(wl.p_logits, 8, dim=1).indices
    for b in range(8):
        assert set(wl.draft_tokens[b].tolist()) <= set(top[b].tolist())


def test_config3_is_zipf_shaped_and_scaled():
    wl = W.config3(batch=2, V=20000)
    assert abs(wl.temp_target - 0.7) < 1e-7 and wl.temp_draft == 1.0 and wl.n == 8 and wl.topk == 50
    srt = torch.sort(wl.q_logits[0], descending=True).values
    # rank-1 logit sits about ln(V) above the median-rank logit
    assert 5.0 < float(srt[0] - srt[10000]) < 14.0


def test_config5_is_bf16_with_overlapping_heads():
    wl = W.config5(batch=2, V=8192, head=200, rows_per_pass=2)
    assert wl.q_logits.dtype == torch.bfloat16 and wl.topk == 100 and wl.n == 16
    tq = set(torch.topk(wl.q_logits[0].float(), 200).indices.tolist())
    tp = set(torch.topk(wl.p_logits[0].float(), 200).indices.tolist())
    # bf16 rounding creates ties at the cut, so allow slack around the 80 % design value
    assert 0.6 <= len(tq & tp) / 200 <= 0.95


def test_config4_cells_have_distinct_seeds():
    a = W.config4(2, 5, 0.25, batch=2, V=1000); b = W.config4(4, 5, 0.25, batch=2, V=1000)
    assert not torch.equal(a.q_logits, b.q_logits)
