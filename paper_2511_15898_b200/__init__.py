"""B200 (sm_100a) implementation of the global-resolution verification rule for
multi-draft speculative sampling: a C-ABI CUDA library plus this thin binding."""
from . import binding
from .binding import (GR_F32, GR_BF16, GR_OK, GR_NOT_CONVERGED, GR_SUPPORT_TOO_LARGE, GR_BAD_LOGITS,
                      GR_DRAFT_OUT_OF_SUPPORT, GR_STALE_PARAMS, GrError, Options, Rule, library_path, load_library,
                      gr_params_bytes, gr_workspace_bytes, gr_solve, gr_solve_static, GR_STATIC_MAX_BATCH, gr_solve_verify, GR_PARTIAL_RULE, gr_alpha_star, alpha_star, gr_verify, gr_read_rule, gr_strerror,
                      solve, verify, solve_verify, read_rule, solve_verify_host, gr_read_slice, read_slice, Slice)

__all__ = [n for n in dir() if not n.startswith("_")]
