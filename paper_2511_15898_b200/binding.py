"""ctypes binding of libgr_b200.so.

Argument marshalling only: every step of the path runs in the CUDA kernels behind
the C interface (include/gr.h).  The low-level functions carry the C names and take
raw device pointers; `solve`, `verify` and `read_rule` accept torch CUDA tensors and
pass their data pointers and the current stream.  There is no CPU fallback: without
the compiled library or without a CUDA device these functions raise.
"""
from __future__ import annotations

import ctypes as C
import dataclasses
import os
from typing import Optional, Tuple

import torch

GR_F32, GR_BF16 = 0, 1
GR_OK, GR_NOT_CONVERGED, GR_SUPPORT_TOO_LARGE, GR_BAD_LOGITS, GR_DRAFT_OUT_OF_SUPPORT, GR_STALE_PARAMS = range(6)
GR_MAX_SUPPORT, GR_MAX_DRAFTS = 128, 32
GR_STATIC_MAX_BATCH = 256
GR_PARTIAL_RULE = 6

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libgr_b200.so")
_lib = None


class GrError(RuntimeError):
    pass


class Options(C.Structure):
    _fields_ = [("tol", C.c_double), ("max_iters", C.c_int), ("quad_step", C.c_double),
                ("scan_done_event", C.c_void_p), ("force_robust", C.c_int), ("tau", C.c_double)]

    def __init__(self, tol: float = 3e-7, max_iters: int = 40, quad_step: float = 0.4, scan_done_event=None,
                 force_robust: int = 0, tau: float = 0.0):
        super().__init__(tol, max_iters, quad_step, scan_done_event, force_robust, tau)


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """dlopen the compiled library (built by paper_2511_15898_b200.build); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise GrError(f"{_LIB_PATH} is missing: build it with `python -m paper_2511_15898_b200.build`")
    lib = C.CDLL(_LIB_PATH)
    vp, ip, fp, dp = C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p
    lib.gr_params_bytes.restype = C.c_size_t
    lib.gr_params_bytes.argtypes = [C.c_int] * 4
    lib.gr_workspace_bytes.restype = C.c_size_t
    lib.gr_workspace_bytes.argtypes = [C.c_int] * 4
    lib.gr_solve.restype = C.c_int
    lib.gr_solve.argtypes = [vp, vp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float, C.c_float, C.c_int,
                             C.POINTER(Options), vp, vp, fp, ip, vp]
    lib.gr_solve_static.restype = C.c_int
    lib.gr_solve_static.argtypes = [vp, vp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float, C.c_float, C.c_int,
                                    C.POINTER(Options), vp, fp, ip, vp]
    lib.gr_solve_verify.restype = C.c_int
    lib.gr_solve_verify.argtypes = [vp, vp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float, C.c_float, C.c_int,
                                    C.POINTER(Options), ip, fp, vp, vp, fp, ip, vp, ip, vp]
    lib.gr_alpha_star.restype = C.c_int
    lib.gr_alpha_star.argtypes = [vp, vp, C.c_int, C.c_int, ip, C.c_int, C.c_int, C.c_float, C.c_float, C.c_int, vp,
                                  fp, ip, vp]
    lib.gr_verify.restype = C.c_int
    lib.gr_verify.argtypes = [vp, ip, fp, C.c_int, ip, vp, ip, vp]
    lib.gr_read_rule.restype = C.c_int
    lib.gr_read_rule.argtypes = [vp, C.c_int, C.c_int, ip, ip, dp, dp, dp, dp, vp]
    lib.gr_read_slice.restype = C.c_int
    lib.gr_read_slice.argtypes = [vp, ip, C.c_int, C.c_int, ip, dp, dp, ip, vp]
    lib.gr_strerror.restype = C.c_char_p
    lib.gr_strerror.argtypes = [C.c_int]
    _lib = lib
    return lib


# ---------------------------------------------------------------- C names, raw pointers

def gr_params_bytes(V: int, n: int, topk: int, batch: int) -> int:
    return int(load_library().gr_params_bytes(V, n, topk, batch))


def gr_workspace_bytes(V: int, n: int, topk: int, batch: int) -> int:
    return int(load_library().gr_workspace_bytes(V, n, topk, batch))


def gr_strerror(code: int) -> str:
    return load_library().gr_strerror(int(code)).decode()


def gr_solve(q_logits: int, p_logits: int, dtype: int, V: int, n: int, topk: int, temp_target: float,
             temp_draft: float, batch: int, opt: Optional[Options], params: int, workspace: int, alpha_star: int,
             status: int, stream: int) -> int:
    return int(load_library().gr_solve(q_logits, p_logits, dtype, V, n, topk, temp_target, temp_draft, batch,
                                       C.byref(opt) if opt is not None else None, params, workspace, alpha_star,
                                       status, stream))


def gr_solve_static(q_logits: int, p_logits: int, dtype: int, V: int, n: int, topk: int, temp_target: float,
                    temp_draft: float, batch: int, opt: Optional[Options], params: int, alpha_star: int, status: int,
                    stream: int) -> int:
    """gr_solve with the scratch inside the library (at most GR_STATIC_MAX_BATCH instances): for callers that
    must not allocate device memory.  Calls that overlap on the GPU share that scratch and race."""
    return int(load_library().gr_solve_static(q_logits, p_logits, dtype, V, n, topk, temp_target, temp_draft, batch,
                                              C.byref(opt) if opt is not None else None, params, alpha_star, status,
                                              stream))


def gr_solve_verify(q_logits: int, p_logits: int, dtype: int, V: int, n: int, topk: int, temp_target: float,
                    temp_draft: float, batch: int, opt: Optional[Options], draft_tokens: int, uniforms: int,
                    params: int, workspace: int, alpha_star: int, out_token: int, out_accepted: int, status: int,
                    stream: int) -> int:
    return int(load_library().gr_solve_verify(q_logits, p_logits, dtype, V, n, topk, temp_target, temp_draft, batch,
                                              C.byref(opt) if opt is not None else None, draft_tokens, uniforms,
                                              params, workspace, alpha_star, out_token, out_accepted, status, stream))


def gr_alpha_star(q_logits: int, p_logits: int, dtype: int, V: int, n_list, topk: int, temp_target: float,
                  temp_draft: float, batch: int, workspace: int, alpha_star: int, status: int, stream: int) -> int:
    ns = (C.c_int * len(n_list))(*[int(x) for x in n_list])
    return int(load_library().gr_alpha_star(q_logits, p_logits, dtype, V, ns, len(n_list), topk, temp_target,
                                            temp_draft, batch, workspace, alpha_star, status, stream))


def gr_verify(params: int, draft_tokens: int, uniforms: int, batch: int, out_token: int, out_accepted: int,
              status: int, stream: int) -> int:
    return int(load_library().gr_verify(params, draft_tokens, uniforms, batch, out_token, out_accepted, status,
                                        stream))


def gr_read_rule(params: int, batch: int, kcap: int, ids: int, block: int, w: int, resid: int, flow: int,
                 header: int, stream: int) -> int:
    return int(load_library().gr_read_rule(params, batch, kcap, ids, block, w, resid, flow, header, stream))


def gr_read_slice(params: int, draft_tokens: int, batch: int, n: int, U: int, pi: int, rho: int, status: int,
                  stream: int) -> int:
    return int(load_library().gr_read_slice(params, draft_tokens, batch, n, U, pi, rho, status, stream))


# ---------------------------------------------------------------- torch tensors

def _check(rc: int, what: str):
    if rc != 0:
        raise GrError(f"{what}: {gr_strerror(rc)} ({rc})")


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return GR_F32
    if t.dtype == torch.bfloat16:
        return GR_BF16
    raise GrError("logits must be float32 or bfloat16")


def _stream() -> int:
    return int(torch.cuda.current_stream().cuda_stream)


def _need_cuda(*ts):
    for t in ts:
        if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous()):
            raise GrError("expected contiguous CUDA tensors")


@dataclasses.dataclass
class Solved:
    """Device-side result of gr_solve: the opaque params block and the per-instance outputs."""
    V: int
    n: int
    topk: int
    batch: int
    params: torch.Tensor       # uint8, opaque
    workspace: torch.Tensor    # uint8, scratch
    alpha_star: torch.Tensor   # [B] float32
    status: torch.Tensor       # [B] int32
    q_logits: torch.Tensor     # kept alive: gr_verify re-reads one chunk of a row on the resample branch


def solve(q_logits: torch.Tensor, p_logits: torch.Tensor, n: int, topk: int, temp_target: float = 1.0,
          temp_draft: float = 1.0, opt: Optional[Options] = None, out: Optional[Solved] = None) -> Solved:
    """gr_solve on torch CUDA tensors ([B, V] float32 or bfloat16), on the current stream."""
    _need_cuda(q_logits, p_logits)
    if q_logits.shape != p_logits.shape or q_logits.dim() != 2 or q_logits.dtype != p_logits.dtype:
        raise GrError("q_logits and p_logits must be [B, V] tensors of one dtype")
    B, V = q_logits.shape
    dev = q_logits.device
    if out is None or out.batch != B or out.V != V or out.n != n or out.topk != topk:
        pbytes = gr_params_bytes(V, n, topk, B)
        wbytes = gr_workspace_bytes(V, n, topk, B)
        if pbytes == 0 or wbytes == 0:
            raise GrError("invalid shape")
        out = Solved(V, n, topk, B,
                     torch.empty(pbytes, dtype=torch.uint8, device=dev),
                     torch.empty(wbytes, dtype=torch.uint8, device=dev),
                     torch.empty(B, dtype=torch.float32, device=dev),
                     torch.empty(B, dtype=torch.int32, device=dev), q_logits)
    out.q_logits = q_logits
    rc = gr_solve(q_logits.data_ptr(), p_logits.data_ptr(), _dtype_code(q_logits), V, n, topk, temp_target,
                  temp_draft, B, opt, out.params.data_ptr(), out.workspace.data_ptr(), out.alpha_star.data_ptr(),
                  out.status.data_ptr(), _stream())
    _check(rc, "gr_solve")
    return out


@dataclasses.dataclass
class Verified:
    token: torch.Tensor      # [B] int32
    accepted: torch.Tensor   # [B] uint8
    status: torch.Tensor     # [B] int32


def verify(solved: Solved, draft_tokens: torch.Tensor, uniforms: torch.Tensor,
           out: Optional[Verified] = None) -> Verified:
    """gr_verify on torch CUDA tensors: draft_tokens [B, n] int32, uniforms [B, 2] float32."""
    _need_cuda(draft_tokens, uniforms)
    B = solved.batch
    if draft_tokens.shape != (B, solved.n) or draft_tokens.dtype != torch.int32:
        raise GrError("draft_tokens must be [B, n] int32")
    if uniforms.shape != (B, 2) or uniforms.dtype != torch.float32:
        raise GrError("uniforms must be [B, 2] float32")
    dev = draft_tokens.device
    if out is None or out.token.shape[0] != B:
        out = Verified(torch.empty(B, dtype=torch.int32, device=dev), torch.empty(B, dtype=torch.uint8, device=dev),
                       torch.empty(B, dtype=torch.int32, device=dev))
    rc = gr_verify(solved.params.data_ptr(), draft_tokens.data_ptr(), uniforms.data_ptr(), B, out.token.data_ptr(),
                   out.accepted.data_ptr(), out.status.data_ptr(), _stream())
    _check(rc, "gr_verify")
    return out


def alpha_star(q_logits: torch.Tensor, p_logits: torch.Tensor, n_list, topk: int, temp_target: float = 1.0,
               temp_draft: float = 1.0) -> Tuple[torch.Tensor, torch.Tensor]:
    """gr_alpha_star on torch CUDA tensors: ([B, len(n_list)] float32 optimal acceptances, [B] int32 status)."""
    _need_cuda(q_logits, p_logits)
    if q_logits.shape != p_logits.shape or q_logits.dim() != 2 or q_logits.dtype != p_logits.dtype:
        raise GrError("q_logits and p_logits must be [B, V] tensors of one dtype")
    B, V = q_logits.shape
    dev = q_logits.device
    wbytes = gr_workspace_bytes(V, 1, topk, B)
    if wbytes == 0:
        raise GrError("invalid shape")
    ws = torch.empty(wbytes, dtype=torch.uint8, device=dev)
    out = torch.empty((B, len(n_list)), dtype=torch.float32, device=dev)
    st = torch.empty(B, dtype=torch.int32, device=dev)
    rc = gr_alpha_star(q_logits.data_ptr(), p_logits.data_ptr(), _dtype_code(q_logits), V, n_list, topk, temp_target,
                       temp_draft, B, ws.data_ptr(), out.data_ptr(), st.data_ptr(), _stream())
    _check(rc, "gr_alpha_star")
    return out, st


def solve_verify(q_logits: torch.Tensor, p_logits: torch.Tensor, draft_tokens: torch.Tensor, uniforms: torch.Tensor,
                 topk: int, temp_target: float = 1.0, temp_draft: float = 1.0, opt: Optional[Options] = None,
                 out: Optional[Tuple[Solved, Verified]] = None) -> Tuple[Solved, Verified]:
    """gr_solve_verify on torch CUDA tensors: one call, the solve kernel finishes every instance with its draw.
    The returned Solved carries alpha* and the params block (partial where a system was skipped); the Verified's
    status is what gr_verify would report."""
    _need_cuda(q_logits, p_logits, draft_tokens, uniforms)
    if q_logits.shape != p_logits.shape or q_logits.dim() != 2 or q_logits.dtype != p_logits.dtype:
        raise GrError("q_logits and p_logits must be [B, V] tensors of one dtype")
    B, V = q_logits.shape
    if draft_tokens.dim() != 2 or draft_tokens.shape[0] != B or draft_tokens.dtype != torch.int32:
        raise GrError("draft_tokens must be [B, n] int32")
    n = int(draft_tokens.shape[1])
    if uniforms.shape != (B, 2) or uniforms.dtype != torch.float32:
        raise GrError("uniforms must be [B, 2] float32")
    dev = q_logits.device
    sv, vf = out if out is not None else (None, None)
    if sv is None or sv.batch != B or sv.V != V or sv.n != n or sv.topk != topk:
        pbytes = gr_params_bytes(V, n, topk, B)
        wbytes = gr_workspace_bytes(V, n, topk, B)
        if pbytes == 0 or wbytes == 0:
            raise GrError("invalid shape")
        sv = Solved(V, n, topk, B, torch.empty(pbytes, dtype=torch.uint8, device=dev),
                    torch.empty(wbytes, dtype=torch.uint8, device=dev),
                    torch.empty(B, dtype=torch.float32, device=dev),
                    torch.empty(B, dtype=torch.int32, device=dev), q_logits)
        vf = None
    if vf is None or vf.token.shape[0] != B:
        vf = Verified(torch.empty(B, dtype=torch.int32, device=dev), torch.empty(B, dtype=torch.uint8, device=dev),
                      sv.status)
    sv.q_logits = q_logits
    vf.status = sv.status
    rc = gr_solve_verify(q_logits.data_ptr(), p_logits.data_ptr(), _dtype_code(q_logits), V, n, topk, temp_target,
                         temp_draft, B, opt, draft_tokens.data_ptr(), uniforms.data_ptr(), sv.params.data_ptr(),
                         sv.workspace.data_ptr(), sv.alpha_star.data_ptr(), vf.token.data_ptr(),
                         vf.accepted.data_ptr(), sv.status.data_ptr(), _stream())
    _check(rc, "gr_solve_verify")
    return sv, vf


@dataclasses.dataclass
class Rule:
    """The verification rule copied out of a params block (host tensors), support in ratio order."""
    ids: torch.Tensor     # [B, kcap] int32, -1 padded
    block: torch.Tensor   # [B, kcap] int32: -1 on H*, else block number from the lowest ratio; -2 padding
    w: torch.Tensor       # [B, kcap] float64 exp(alpha)
    resid: torch.Tensor   # [B, kcap] float64 outer residual
    flow: torch.Tensor    # [B, kcap] float64 p_i
    k: torch.Tensor       # [B]
    jstar: torch.Tensor
    nblocks: torch.Tensor
    alpha_star: torch.Tensor   # [B] float64
    gnorm: torch.Tensor
    iters: torch.Tensor        # gradient evaluations spent
    lse_target: torch.Tensor
    status: torch.Tensor
    gnorm_predicted: torch.Tensor = None   # [B] bool: the norm of some system was predicted from its last Newton step


def read_rule(solved: Solved) -> Rule:
    B = solved.batch
    kfull = solved.V if (solved.topk <= 0 or solved.topk >= solved.V) else solved.topk
    kcap = max(1, min(kfull, GR_MAX_SUPPORT))
    dev = solved.params.device
    ids = torch.empty(B, kcap, dtype=torch.int32, device=dev)
    blk = torch.empty(B, kcap, dtype=torch.int32, device=dev)
    w = torch.empty(B, kcap, dtype=torch.float64, device=dev)
    r = torch.empty(B, kcap, dtype=torch.float64, device=dev)
    p = torch.empty(B, kcap, dtype=torch.float64, device=dev)
    hd = torch.empty(B, 8, dtype=torch.float64, device=dev)
    rc = gr_read_rule(solved.params.data_ptr(), B, kcap, ids.data_ptr(), blk.data_ptr(), w.data_ptr(), r.data_ptr(),
                      p.data_ptr(), hd.data_ptr(), _stream())
    _check(rc, "gr_read_rule")
    hd = hd.cpu()
    return Rule(ids.cpu(), blk.cpu(), w.cpu(), r.cpu(), p.cpu(), hd[:, 0].long(), hd[:, 1].long(), hd[:, 2].long(),
                hd[:, 3], hd[:, 4], hd[:, 5].long() & 0xffff, hd[:, 6], hd[:, 7].long(), (hd[:, 5].long() >> 16) & 1 == 1)


@dataclasses.dataclass
class Slice:
    """pi(.|omega) per instance as the verification code computes it (host tensors)."""
    U: torch.Tensor        # [B, n] int32: drafted token s, -1 for a repeat
    pi: torch.Tensor       # [B, n] float64
    rho: torch.Tensor      # [B] float64 mass of the resample segment
    status: torch.Tensor   # [B] int32


def read_slice(solved: Solved, draft_tokens: torch.Tensor) -> Slice:
    """gr_read_slice on torch CUDA tensors."""
    _need_cuda(draft_tokens)
    B, n = solved.batch, solved.n
    if draft_tokens.shape != (B, n) or draft_tokens.dtype != torch.int32:
        raise GrError("draft_tokens must be [B, n] int32")
    dev = draft_tokens.device
    U = torch.empty(B, n, dtype=torch.int32, device=dev)
    pi = torch.empty(B, n, dtype=torch.float64, device=dev)
    rho = torch.empty(B, dtype=torch.float64, device=dev)
    st = torch.empty(B, dtype=torch.int32, device=dev)
    rc = gr_read_slice(solved.params.data_ptr(), draft_tokens.data_ptr(), B, n, U.data_ptr(), pi.data_ptr(),
                       rho.data_ptr(), st.data_ptr(), _stream())
    _check(rc, "gr_read_slice")
    return Slice(U.cpu(), pi.cpu(), rho.cpu(), st.cpu())


def solve_verify_host(q_logits: torch.Tensor, p_logits: torch.Tensor, draft_tokens: torch.Tensor,
                      uniforms: torch.Tensor, n: int, topk: int, temp_target: float = 1.0, temp_draft: float = 1.0,
                      opt: Optional[Options] = None, device="cuda:0", state: Optional[dict] = None):
    """The whole path for HOST tensors (pinned or pageable): copies the inputs to the device, runs gr_solve and
    gr_verify on the current stream and copies token / accepted / alpha* back.  `state` (a dict the caller keeps)
    lets repeated calls reuse the device buffers."""
    st = state if state is not None else {}
    dev = torch.device(device)

    def dev_buf(name, src):
        buf = st.get(name)
        if buf is None or buf.shape != src.shape or buf.dtype != src.dtype:
            buf = torch.empty(src.shape, dtype=src.dtype, device=dev)
            st[name] = buf
        buf.copy_(src, non_blocking=True)
        return buf

    q = dev_buf("q", q_logits); p = dev_buf("p", p_logits)
    tk = dev_buf("tk", draft_tokens); un = dev_buf("un", uniforms)
    st["solved"] = solve(q, p, n, topk, temp_target, temp_draft, opt, st.get("solved"))
    st["verified"] = verify(st["solved"], tk, un, st.get("verified"))
    v = st["verified"]
    return v.token.cpu(), v.accepted.cpu(), st["solved"].alpha_star.cpu(), v.status.cpu()
