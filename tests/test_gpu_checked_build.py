"""The bounds-checked build of the library (-DGR_CHECK), the stand-in for a memory checker on machines where none
may run: every pointer into shared memory, the workspace records and the params block carries its extent, an access
outside it is skipped and reported as status GR_CHECK_FAILED.  The test runs small cases of every kernel family
through that build in a child process (the binding holds one library per process) and expects no such status and the
same results as the regular build; a self-test of the checked pointer shows that it does catch and skip."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu

CHILD = r"""
import json, sys, ctypes
sys.path.insert(0, %(root)r)
import torch
import paper_2511_15898_b200.binding as Bn
from paper_2511_15898_b200.build import build_library
checked = %(checked)d
Bn._LIB_PATH = build_library(check=bool(checked))
import paper_2511_15898_b200 as G
from paper_2511_15898_b200 import workloads as W
lib = G.load_library()
out = {"cases": []}
if checked:
    buf = torch.zeros(4, dtype=torch.int32, device="cuda")
    lib.gr_check_selftest.restype = ctypes.c_int
    lib.gr_check_selftest.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
    assert lib.gr_check_selftest(buf.data_ptr(), None) == 0
    torch.cuda.synchronize()
    out["selftest"] = buf.cpu().tolist()
cases = [("config1", W.config1(batch=16, device="cuda"), None),
         ("config2 V=5000", W.config2(batch=8, device="cuda", V=5000), None),
         ("support 80, n=6", W.config3(batch=4, device="cuda", seed=3100, V=20000, n=6, topk=80), None),
         ("support 128, n=16", W.config3(batch=3, device="cuda", seed=3101, V=20000, n=16, topk=128), None),
         ("ragged V=1031", W.config4(3, 6, 1.0, batch=5, device="cuda", V=1031, seed=77), None),
         ("ragged V=4099 n=32 (robust kernel)", W.config4(32, 20, 1.0, batch=3, device="cuda", V=4099, seed=78), None),
         ("headline shape, robust kernel", W.config3(batch=3, device="cuda", seed=3102), G.Options(force_robust=1)),
         ("headline shape, tau=0.05", W.config3(batch=4, device="cuda", seed=3103), G.Options(tau=0.05)),
         ("whole vocabulary V=5000", W.config4(4, 0, 1.0, batch=3, device="cuda", V=5000, seed=99), None),
         ("whole vocabulary V=50257 (bucket search)", W.config4(8, 0, 1.0, batch=2, device="cuda", seed=98), None),
         ("whole vocabulary V=5000 (sort)", W.config4(4, 0, 1.0, batch=2, device="cuda", V=5000, seed=97),
          G.Options(force_robust=1)),
         ("bf16 V=9001", W.config5(batch=4, device="cuda", V=9001, rows_per_pass=4), None)]
for name, wl, opt in cases:
    s = G.solve(wl.q_logits, wl.p_logits, wl.n, wl.topk, wl.temp_target, wl.temp_draft, opt)
    v = G.verify(s, wl.draft_tokens, wl.uniforms)
    sl = G.read_slice(s, wl.draft_tokens)
    sv, vf = G.solve_verify(wl.q_logits, wl.p_logits, wl.draft_tokens, wl.uniforms, wl.topk, wl.temp_target,
                            wl.temp_draft, opt)
    torch.cuda.synchronize()
    out["cases"].append({"name": name, "solve_status": s.status.cpu().tolist(), "verify_status": v.status.cpu().tolist(),
                         "fused_status": vf.status.cpu().tolist(), "tokens": v.token.cpu().tolist(),
                         "fused_tokens": vf.token.cpu().tolist(),
                         "alpha": [round(float(x), 7) for x in s.alpha_star.cpu().tolist()]})
print("RESULT " + json.dumps(out))
"""


def _run(checked: int):
    code = CHILD % {"root": ROOT, "checked": checked}
    res = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=1500)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    line = [ln for ln in res.stdout.splitlines() if ln.startswith("RESULT ")][-1]
    return json.loads(line[len("RESULT "):])


def test_checked_build_reports_nothing_and_agrees_with_the_regular_build():
    chk = _run(1)
    ref = _run(0)
    # the checked pointer itself: two of six accesses (indices -1 and 4) skipped and flagged, reads there gave 0,
    # the array is untouched
    assert chk["selftest"] == [2, 6, 0, 6], chk["selftest"]
    GR_CHECK_FAILED = 7
    for a, b in zip(chk["cases"], ref["cases"]):
        assert a["name"] == b["name"]
        for key in ("solve_status", "verify_status", "fused_status"):
            assert GR_CHECK_FAILED not in a[key], (a["name"], key, a[key])
        assert a["solve_status"] == b["solve_status"] and a["verify_status"] == b["verify_status"], a["name"]
        assert a["tokens"] == b["tokens"] and a["fused_tokens"] == b["fused_tokens"], a["name"]
        assert a["alpha"] == b["alpha"] or all(abs(x - y) <= 1e-6 or (x != x and y != y)
                                               for x, y in zip(a["alpha"], b["alpha"])), a["name"]
