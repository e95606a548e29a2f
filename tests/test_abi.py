"""Host-side checks that need no GPU: the library builds for sm_100a, loads, exports every
symbol the header declares, and rejects bad arguments before launching anything."""
import ctypes as C
import os
import re

import pytest

import paper_2511_15898_b200 as G
from paper_2511_15898_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_library()
    return G.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "gr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gr_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert {"gr_solve", "gr_verify", "gr_params_bytes", "gr_workspace_bytes", "gr_read_rule",
            "gr_strerror"} <= set(names)
    for nm in names:
        assert hasattr(lib, nm), nm


def test_size_queries(lib):
    assert G.gr_params_bytes(128256, 8, 50, 1024) % 16 == 0
    per = G.gr_params_bytes(128256, 8, 50, 1)
    assert G.gr_params_bytes(128256, 8, 50, 1024) == 1024 * per
    # header + 32 bytes per support slot + 8 bytes per 1024-element chunk
    assert per >= 96 + 32 * 50 + 8 * 126
    assert G.gr_workspace_bytes(128256, 8, 50, 1024) > 0
    # invalid shapes
    assert G.gr_params_bytes(0, 8, 50, 4) == 0
    assert G.gr_params_bytes(16, 0, 0, 4) == 0
    assert G.gr_params_bytes(16, 33, 0, 4) == 0
    assert G.gr_workspace_bytes(16, 2, 0, -1) == 0
    # whole-vocabulary support beyond the capacity still gets a header and a chunk table
    assert G.gr_params_bytes(50257, 4, 0, 2) >= 2 * (96 + 8 * 50)


def test_argument_errors_are_reported_before_any_launch(lib):
    A = 1 << 20   # any 16-byte aligned non-null address: nothing is dereferenced on these paths
    ok = dict(q=A, p=A, dtype=G.GR_F32, V=1000, n=4, topk=8, tt=1.0, td=1.0, batch=2)

    def call(**kw):
        a = dict(ok); a.update(kw)
        return G.gr_solve(a["q"], a["p"], a["dtype"], a["V"], a["n"], a["topk"], a["tt"], a["td"], a["batch"],
                          a.get("opt"), A, A, A, A, 0)

    assert call(V=0) == -1
    assert call(n=0) == -1 and call(n=33) == -1
    assert call(batch=-1) == -1
    assert call(tt=0.0) == -1 and call(td=-1.0) == -1 and call(tt=float("nan")) == -1
    assert call(dtype=7) == -1
    assert call(q=0) == -2
    assert call(q=A + 4) == -3
    assert call(opt=G.Options(tol=0.0)) == -1
    assert call(opt=G.Options(quad_step=5.0)) == -1
    assert call(opt=G.Options(max_iters=0)) == -1
    assert call(opt=G.Options(tau=-1e-3)) == -1 and call(opt=G.Options(tau=1.5)) == -1
    assert call(opt=G.Options(tau=float("nan"))) == -1
    assert call(V=100000, topk=500) == -5        # truncated support beyond GR_MAX_SUPPORT
    assert call(batch=0) == 0                    # an empty batch is a no-op
    assert G.gr_verify(0, A, A, 2, A, A, A, 0) == -2
    assert G.gr_verify(A, A, A, -1, A, A, A, 0) == -1
    assert G.gr_verify(A, A, A, 0, A, A, A, 0) == 0
    assert G.gr_read_rule(0, 1, 8, 0, 0, 0, 0, 0, 0, 0) == -2
    assert G.gr_read_slice(0, A, 2, 4, A, A, A, A, 0) == -2 and G.gr_read_slice(A, A, 2, 4, 0, A, A, A, 0) == -2
    assert G.gr_read_slice(A, A, 2, 0, A, A, A, A, 0) == -1 and G.gr_read_slice(A, A, -1, 4, A, A, A, A, 0) == -1
    assert G.gr_read_slice(A + 4, A, 2, 4, A, A, A, A, 0) == -3 and G.gr_read_slice(A, A, 0, 4, A, A, A, A, 0) == 0
    # the fused entry: gr_solve's checks plus its own pointers
    def fused(**kw):
        a = dict(ok); a.update(kw)
        return G.gr_solve_verify(a["q"], a["p"], a["dtype"], a["V"], a["n"], a["topk"], a["tt"], a["td"], a["batch"],
                                 None, a.get("draft", A), a.get("uni", A), A, A, A, a.get("tok", A), A, A, 0)
    assert fused(draft=0) == -2 and fused(uni=0) == -2 and fused(tok=0) == -2
    assert fused(V=0) == -1 and fused(q=A + 4) == -3 and fused(batch=0) == 0
    # the acceptance-only entry
    def alpha(ns, **kw):
        a = dict(ok); a.update(kw)
        return G.gr_alpha_star(a["q"], a["p"], a["dtype"], a["V"], ns, a["topk"], a["tt"], a["td"], a["batch"], A, A,
                               A, 0)
    assert alpha([]) == -1 and alpha([0]) == -1 and alpha([33]) == -1 and alpha(list(range(1, 10))) == -1
    assert alpha([2], q=0) == -2 and alpha([2], q=A + 4) == -3 and alpha([2], tt=0.0) == -1
    assert alpha([2], V=100000, topk=500) == -5   # truncated support beyond GR_MAX_SUPPORT
    assert alpha([2, 4], batch=0) == 0


def test_strerror(lib):
    assert G.gr_strerror(0) == "ok"
    for code in (1, 2, 3, 4, 5, 6, -1, -2, -3, -4, -5):
        assert G.gr_strerror(code) not in ("", "unknown code")
    assert G.gr_strerror(99) == "unknown code"


def test_tensor_front_end_refuses_cpu_tensors(lib):
    import torch
    q = torch.zeros(2, 16)
    with pytest.raises(G.GrError):
        G.solve(q, q, 2, 0)
    with pytest.raises(G.GrError):
        G.alpha_star(q, q, [2], 0)
    with pytest.raises(G.GrError):
        G.solve_verify(q, q, torch.zeros(2, 2, dtype=torch.int32), torch.zeros(2, 2), 0)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    import paper_2511_15898_b200.binding as Bn
    monkeypatch.setattr(Bn, "_lib", None)
    monkeypatch.setattr(Bn, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(G.GrError):
        Bn.load_library()
