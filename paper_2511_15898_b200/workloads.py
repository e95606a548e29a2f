"""Seeded synthetic workloads for the multi-draft verification path.

This module only manufactures inputs: target / draft logits with the shapes and
value distributions of the benchmark configurations, the n drafted tokens (what
a draft model's top-k sampler would hand over) and the verification uniforms.
It contains none of the method's arithmetic (no subset selection, residuals,
convex solve or verification rule) and is the only code shared by the CPU
oracle's tests and the CUDA path's tests / benchmark.

Naming: ``q_logits`` are the TARGET model's logits and ``p_logits`` the DRAFT
model's, as in the library's C interface (the paper uses the opposite letters).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import torch


@dataclasses.dataclass
class Workload:
    name: str
    V: int
    n: int
    topk: int            # 0 = full support
    temp_target: float
    temp_draft: float
    q_logits: torch.Tensor      # [B, V] target logits, fp32 or bf16
    p_logits: torch.Tensor      # [B, V] draft logits, same dtype
    draft_tokens: torch.Tensor  # [B, n] int32, i.i.d. draws from the truncated draft distribution
    uniforms: torch.Tensor      # [B, 2] fp32 in [0, 1): verification uniforms (u0, u1)

    def __post_init__(self):
        # the C interface takes the temperatures as float: keep exactly those values, so that every
        # consumer of the workload (CUDA path, CPU oracle) divides by the same numbers
        self.temp_target = float(torch.tensor(self.temp_target, dtype=torch.float32).item())
        self.temp_draft = float(torch.tensor(self.temp_draft, dtype=torch.float32).item())

    @property
    def batch(self) -> int:
        return self.q_logits.shape[0]

    def to(self, device) -> "Workload":
        return dataclasses.replace(
            self,
            q_logits=self.q_logits.to(device),
            p_logits=self.p_logits.to(device),
            draft_tokens=self.draft_tokens.to(device),
            uniforms=self.uniforms.to(device),
        )

    def rows(self, idx) -> "Workload":
        """Sub-batch made of the given instance indices (kept on the same device)."""
        idx = torch.as_tensor(idx, device=self.q_logits.device, dtype=torch.long)
        return dataclasses.replace(
            self,
            q_logits=self.q_logits[idx].contiguous(),
            p_logits=self.p_logits[idx].contiguous(),
            draft_tokens=self.draft_tokens[idx].contiguous(),
            uniforms=self.uniforms[idx].contiguous(),
        )


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _random_perm_rows(B: int, V: int, g: torch.Generator, device) -> torch.Tensor:
    """One uniformly random permutation of 0..V-1 per row (rank -> token id)."""
    keys = torch.rand(B, V, generator=g, device=device)
    return torch.argsort(keys, dim=1)


def _zipf_rows(B, V, exponent, noise_std, g, device, perm: Optional[torch.Tensor] = None):
    """Logit of the token holding rank r is -exponent*ln(r) + N(0, noise_std^2);
    ranks are laid over token ids by a random permutation per row."""
    ranks = torch.arange(1, V + 1, device=device, dtype=torch.float32)
    by_rank = -exponent * torch.log(ranks)[None, :] + noise_std * torch.randn(B, V, generator=g, device=device)
    if perm is None:
        perm = _random_perm_rows(B, V, g, device)
    out = torch.empty_like(by_rank)
    out.scatter_(1, perm, by_rank)
    return out, perm


def sample_draft_tokens(p_logits: torch.Tensor, topk: int, temp_draft: float, n: int,
                        g: torch.Generator) -> torch.Tensor:
    """What the draft model's sampler does: keep the `topk` largest draft logits
    (ties: the smaller token id is kept), softmax at `temp_draft` over the kept
    ids, and draw n i.i.d. tokens by inverse CDF over the kept ids in ascending
    id order, one uniform per draw.  topk == 0 or >= V keeps every id."""
    B, V = p_logits.shape
    dev = p_logits.device
    x = p_logits.to(torch.float32)
    k = V if (topk <= 0 or topk >= V) else topk
    if k < V:
        # stable descending sort: equal logits keep ascending id order
        _, order = torch.sort(x, dim=1, descending=True, stable=True)
        ids = torch.sort(order[:, :k], dim=1).values
    else:
        ids = torch.arange(V, device=dev)[None, :].expand(B, V)
    z = torch.gather(x, 1, ids).to(torch.float64) / float(temp_draft)
    prob = torch.softmax(z, dim=1)
    cdf = torch.cumsum(prob, dim=1)
    u = torch.rand(B, n, generator=g, device=dev, dtype=torch.float64)
    pos = torch.searchsorted(cdf, u * cdf[:, -1:], right=True).clamp_(max=k - 1)
    return torch.gather(ids, 1, pos).to(torch.int32)


def _finish(name, V, n, topk, Tt, Td, q, p, g, dtype=torch.float32) -> Workload:
    q = q.to(dtype).contiguous()
    p = p.to(dtype).contiguous()
    toks = sample_draft_tokens(p, topk, Td, n, g)
    B = q.shape[0]
    uni = torch.rand(B, 2, generator=g, device=q.device, dtype=torch.float32)
    return Workload(name, V, n, topk, Tt, Td, q, p, toks.contiguous(), uni.contiguous())


def config1(batch: int = 64, device="cpu", seed: int = 1000) -> Workload:
    """Tiny check case: V=16, n=2, full-support draft, N(0,2^2) target logits,
    draft = target + N(0,0.5^2), temperature 1."""
    V, n = 16, 2
    g = _gen(seed, device)
    q = 2.0 * torch.randn(batch, V, generator=g, device=device)
    p = q + 0.5 * torch.randn(batch, V, generator=g, device=device)
    return _finish("config1", V, n, 0, 1.0, 1.0, q, p, g)


def config2(batch: int = 256, device="cpu", seed: int = 2000, V: int = 32000) -> Workload:
    """V=32000, n=4, top-8 draft; Zipf(1.1) + N(0,1) target, draft = target + N(0,1)."""
    n, k = 4, 8
    g = _gen(seed, device)
    q, _ = _zipf_rows(batch, V, 1.1, 1.0, g, device)
    p = q + torch.randn(batch, V, generator=g, device=device)
    return _finish("config2", V, n, k, 1.0, 1.0, q, p, g)


def config3(batch: int = 1024, device="cpu", seed: int = 3000, V: int = 128256,
            n: int = 8, topk: int = 50) -> Workload:
    """Headline: V=128256, n=8, top-50 draft; Zipf(1.0)+N(0,0.5^2) target, draft =
    target + N(0,0.75^2); target temperature 0.7, draft temperature 1.0."""
    g = _gen(seed, device)
    q, _ = _zipf_rows(batch, V, 1.0, 0.5, g, device)
    p = q + 0.75 * torch.randn(batch, V, generator=g, device=device)
    return _finish("config3", V, n, topk, 0.7, 1.0, q, p, g)


CONFIG4_N = (2, 4, 8, 16, 32)
CONFIG4_K = (5, 20, 0)          # 0 = full vocabulary
CONFIG4_SIGMA = (0.25, 1.0, 2.0)


def config4(n: int, topk: int, sigma: float, batch: int = 512, device="cpu",
            seed: Optional[int] = None, V: int = 50257) -> Workload:
    """n-sweep cell: V=50257, N(0,3^2) target logits, draft = target + N(0,sigma^2)."""
    if seed is None:
        cell = (CONFIG4_N.index(n) * len(CONFIG4_K) + CONFIG4_K.index(topk)) * len(CONFIG4_SIGMA) \
            + CONFIG4_SIGMA.index(sigma)
        seed = 4000 + cell
    g = _gen(seed, device)
    q = 3.0 * torch.randn(batch, V, generator=g, device=device)
    p = q + sigma * torch.randn(batch, V, generator=g, device=device)
    return _finish(f"config4[n={n},k={topk or 'V'},sigma={sigma}]", V, n, topk, 1.0, 1.0, q, p, g)


def config5(batch: int = 4096, device="cpu", seed: int = 5000, V: int = 152064,
            n: int = 16, topk: int = 100, head: int = 1000, overlap: float = 0.8,
            rows_per_pass: int = 256) -> Workload:
    """Large serving batch: V=152064, n=16, top-100 draft, bf16 logits.  Target is
    Zipf(1.2)+N(0,1); the draft is an independent Zipf draw of the same law whose
    `head` best-ranked ids share `overlap` of the target's `head` best-ranked ids.
    Target temperature 1.0, draft temperature 0.8."""
    g = _gen(seed, device)
    head = min(head, V // 2)
    keep = int(round(overlap * head))
    qs, ps = [], []
    for lo in range(0, batch, rows_per_pass):
        b = min(rows_per_pass, batch - lo)
        q, _ = _zipf_rows(b, V, 1.2, 1.0, g, device)
        # ids of the target row ordered by decreasing logit (value rank -> token id)
        order_q = torch.argsort(q, dim=1, descending=True, stable=True)
        # draft ranking by value: its `head` largest logits sit on `keep` ids drawn from
        # the target's `head` largest and head-keep ids drawn from the rest, in random order.
        k_head = torch.rand(b, head, generator=g, device=device)
        k_tail = torch.rand(b, V - head, generator=g, device=device)
        head_sel = torch.argsort(k_head, dim=1)          # random order of the target's head ranks
        tail_sel = torch.argsort(k_tail, dim=1) + head   # random order of the target's tail ranks
        first = torch.cat([head_sel[:, :keep], tail_sel[:, : head - keep]], dim=1)
        rest = torch.cat([head_sel[:, keep:], tail_sel[:, head - keep:]], dim=1)
        first = torch.gather(first, 1, torch.argsort(torch.rand(b, head, generator=g, device=device), dim=1))
        rest = torch.gather(rest, 1, torch.argsort(torch.rand(b, V - head, generator=g, device=device), dim=1))
        rank_of_target_rank = torch.cat([first, rest], dim=1)   # draft value rank -> target value rank
        perm_p = torch.gather(order_q, 1, rank_of_target_rank)  # draft value rank -> token id
        ranks = torch.arange(1, V + 1, device=device, dtype=torch.float32)
        vals = -1.2 * torch.log(ranks)[None, :] + torch.randn(b, V, generator=g, device=device)
        vals = torch.sort(vals, dim=1, descending=True).values  # an independent draw of the same law, by value rank
        p = torch.empty_like(vals)
        p.scatter_(1, perm_p, vals)
        qs.append(q.to(torch.bfloat16))
        ps.append(p.to(torch.bfloat16))
    q = torch.cat(qs, 0)
    p = torch.cat(ps, 0)
    return _finish("config5", V, n, topk, 1.0, 0.8, q, p, g, dtype=torch.bfloat16)


def logits_to_f64(t: torch.Tensor):
    """Exact upcast of fp32 / bf16 logits to a float64 numpy array on the host."""
    return t.detach().to("cpu").to(torch.float64).numpy()
