"""ctypes binding of libziplm.so: argument marshalling only, every step runs in the CUDA kernels.

Function names and arguments mirror ``include/ziplm.h``.  Tensors are torch CUDA tensors; they
are used as device buffers (``data_ptr``) and the current torch stream is passed down.  There is
no fallback: if the shared library is missing or was not built, importing a function works but
calling it raises :class:`ZiplmError`.
"""
from __future__ import annotations

import ctypes
import enum
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None


class Status(enum.IntEnum):
    OK = 0
    ERR_INVALID_ARG = 1
    ERR_WORKSPACE = 2
    ERR_NOT_PD = 3
    ERR_NONFINITE = 4
    ERR_TIMEOUT = 5
    ERR_CUDA = 6
    ERR_UNSUPPORTED = 7


F32, BF16, F16 = 0, 1, 2
_DTYPES = {torch.float32: F32, torch.bfloat16: BF16, torch.float16: F16}


class ZiplmError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = Status(status) if status in Status._value2member_map_ else status
        super().__init__(f"{where}: {status_string(status)}")


def lib_path() -> str:
    return os.path.join(_HERE, "libziplm.so")


def load_library() -> ctypes.CDLL:
    """Load libziplm.so (built by ``python -m paper_2302_04089_b200.build``) and type its symbols."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = lib_path()
    if not os.path.exists(path):
        raise ZiplmError(Status.ERR_CUDA, f"{path} is missing -- run paper_2302_04089_b200/build.py; "
                                          "there is no CPU fallback")
    lib = ctypes.CDLL(path)
    c_int, c_ll, c_f, c_sz, vp = (ctypes.c_int, ctypes.c_longlong, ctypes.c_float, ctypes.c_size_t,
                                  ctypes.c_void_p)
    lib.ziplm_status_string.restype = ctypes.c_char_p
    lib.ziplm_status_string.argtypes = [c_int]
    lib.ziplm_hessian_workspace_bytes.restype = c_sz
    lib.ziplm_hessian_workspace_bytes.argtypes = [c_int, c_int, c_ll, c_int]
    lib.ziplm_hessian_accumulate.restype = c_int
    lib.ziplm_hessian_accumulate.argtypes = [vp, vp, c_int, c_int, c_int, c_ll, c_ll, c_f, c_f, vp,
                                             c_sz, vp]
    lib.ziplm_hessian_tokens_workspace_bytes.restype = c_sz
    lib.ziplm_hessian_tokens_workspace_bytes.argtypes = [c_int, c_int, c_ll, c_int]
    lib.ziplm_hessian_accumulate_tokens.restype = c_int
    lib.ziplm_hessian_accumulate_tokens.argtypes = [vp, vp, c_int, c_int, c_int, c_ll, c_ll, c_f, c_f,
                                                    vp, c_sz, vp]
    lib.ziplm_inverse_workspace_bytes.restype = c_sz
    lib.ziplm_inverse_workspace_bytes.argtypes = [c_int, c_int]
    lib.ziplm_damped_inverse.restype = c_int
    lib.ziplm_damped_inverse.argtypes = [vp, c_int, c_int, c_f, vp, vp, vp, c_sz, vp]
    lib.ziplm_damped_inverse_noalloc.restype = c_int
    lib.ziplm_damped_inverse_noalloc.argtypes = [vp, c_int, c_int, c_f, vp, vp, vp]
    lib.ziplm_prune_workspace_bytes.restype = c_sz
    lib.ziplm_prune_workspace_bytes.argtypes = [c_int, c_int, c_int, c_int, c_int]
    lib.ziplm_prune_layers.restype = c_int
    lib.ziplm_prune_layers.argtypes = [vp, vp, c_int, c_int, c_int, c_int, c_f,
                                       ctypes.POINTER(c_int), c_int, vp, vp, vp, vp, vp, vp, vp,
                                       c_sz, vp]
    lib.ziplm_kept_structures.restype = c_int
    lib.ziplm_kept_structures.argtypes = [vp, c_int, c_int, c_int, vp, vp, vp]
    lib.ziplm_gather_columns.restype = c_int
    lib.ziplm_gather_columns.argtypes = [vp, c_ll, c_ll, vp, c_int, c_int, c_int, c_int, c_int, vp, vp]
    lib.ziplm_gather_rows.restype = c_int
    lib.ziplm_gather_rows.argtypes = [vp, c_ll, c_ll, vp, c_int, c_int, c_int, c_int, c_int, vp, vp]
    lib.ziplm_select_workspace_bytes.restype = c_sz
    lib.ziplm_select_workspace_bytes.argtypes = [c_int, c_int, c_int]
    lib.ziplm_select_levels.restype = c_int
    lib.ziplm_select_levels.argtypes = [vp, vp, vp, vp, c_int, c_int, vp, c_int, ctypes.c_double, c_int,
                                        vp, vp, vp, vp, vp, c_sz, vp]
    lib.ziplm_search_workspace_bytes.restype = c_sz
    lib.ziplm_search_workspace_bytes.argtypes = [c_int, c_int, c_int]
    lib.ziplm_search_levels.restype = c_int
    lib.ziplm_search_levels.argtypes = [vp, vp, vp, vp, c_int, c_int, vp, vp, vp, c_int, c_int, vp, vp,
                                        c_int, vp, vp, vp, vp, vp, vp, c_sz, vp]
    lib.ziplm_set_option.restype = c_int
    lib.ziplm_set_option.argtypes = [c_int, c_int]
    lib.ziplm_get_option.restype = c_int
    lib.ziplm_get_option.argtypes = [c_int]
    lib.ziplm_launch_count.restype = ctypes.c_longlong
    lib.ziplm_launch_count.argtypes = []
    lib.ziplm_profile_begin.restype = c_int
    lib.ziplm_profile_begin.argtypes = []
    lib.ziplm_profile_end.restype = c_int
    lib.ziplm_profile_end.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.POINTER(c_ll), c_int]
    lib.ziplm_profile_phase_count.restype = c_int
    lib.ziplm_profile_phase_count.argtypes = []
    lib.ziplm_profile_phase_name.restype = ctypes.c_char_p
    lib.ziplm_profile_phase_name.argtypes = [c_int]
    _LIB = lib
    return lib


def status_string(status: int) -> str:
    try:
        return load_library().ziplm_status_string(int(status)).decode()
    except ZiplmError:
        return f"status {int(status)}"


def _stream_ptr(t: torch.Tensor) -> int:
    return torch.cuda.current_stream(t.device).cuda_stream


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _check(t: torch.Tensor, dtype, name: str):
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA tensor of dtype {dtype}")


def _workspace(nbytes: int, device) -> torch.Tensor:
    # torch's caching allocator returns 512-byte aligned blocks
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def hessian_workspace_bytes(L: int, d: int, n_tokens: int, x_dtype: int) -> int:
    return int(load_library().ziplm_hessian_workspace_bytes(L, d, n_tokens, x_dtype))


def hessian_tokens_workspace_bytes(L: int, d: int, n_tokens: int, a_dtype: int) -> int:
    return int(load_library().ziplm_hessian_tokens_workspace_bytes(L, d, n_tokens, a_dtype))


def inverse_workspace_bytes(L: int, d: int) -> int:
    return int(load_library().ziplm_inverse_workspace_bytes(L, d))


def prune_workspace_bytes(L: int, d_row: int, d_col: int, group_size: int, n_levels: int) -> int:
    return int(load_library().ziplm_prune_workspace_bytes(L, d_row, d_col, group_size, n_levels))


def hessian_accumulate(X: torch.Tensor, H: Optional[torch.Tensor] = None, alpha: float = 2.0,
                       beta: float = 0.0, workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """H = beta * H + alpha * X X^T per layer.  X [L, d, N] fp32, bf16 or fp16 (tokens contiguous)."""
    lib = load_library()
    if X.dim() != 3 or not X.is_cuda or X.stride(2) != 1 and X.shape[2] > 1:
        raise ValueError("X must be a CUDA tensor [L, d, N] with contiguous tokens")
    if X.dtype not in _DTYPES:
        raise ValueError("X must be fp32, bf16 or fp16")
    L, d, N = X.shape
    if X.stride(0) != d * X.stride(1):
        raise ValueError("layers of X must be evenly pitched")
    ldx = X.stride(1) if N > 0 else max(N, 1)
    dt = _DTYPES[X.dtype]
    if H is None:
        H = torch.zeros(L, d, d, dtype=torch.float32, device=X.device)
        beta = 0.0
    _check(H, torch.float32, "H")
    need = hessian_workspace_bytes(L, d, N, dt)
    if workspace is None:
        workspace = _workspace(need, X.device)
    with torch.cuda.device(X.device):
        st = lib.ziplm_hessian_accumulate(H.data_ptr(), X.data_ptr(), dt, L, d, N, ldx, alpha, beta,
                                          workspace.data_ptr(), workspace.numel(), _stream_ptr(X))
    if st != 0:
        raise ZiplmError(st, "ziplm_hessian_accumulate")
    return H


def hessian_accumulate_tokens(A: torch.Tensor, H: Optional[torch.Tensor] = None, alpha: float = 2.0,
                              beta: float = 0.0,
                              workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """H = beta * H + alpha * A^T A per layer.  A [L, N, d] fp32, bf16 or fp16, one token per row
    (features contiguous); the row pitch may exceed d.  See ziplm_hessian_accumulate_tokens."""
    lib = load_library()
    if A.dim() != 3 or not A.is_cuda or A.stride(2) != 1 and A.shape[2] > 1:
        raise ValueError("A must be a CUDA tensor [L, N, d] with contiguous features")
    if A.dtype not in _DTYPES:
        raise ValueError("A must be fp32, bf16 or fp16")
    L, N, d = A.shape
    lda = A.stride(1) if N > 1 else d
    if L > 1 and N > 0 and A.stride(0) != N * lda:
        raise ValueError("layers of A must be evenly pitched")
    dt = _DTYPES[A.dtype]
    if H is None:
        H = torch.zeros(L, d, d, dtype=torch.float32, device=A.device)
        beta = 0.0
    _check(H, torch.float32, "H")
    need = hessian_tokens_workspace_bytes(L, d, N, dt)
    if workspace is None:
        workspace = _workspace(need, A.device)
    with torch.cuda.device(A.device):
        st = lib.ziplm_hessian_accumulate_tokens(H.data_ptr(), A.data_ptr(), dt, L, d, N, lda, alpha,
                                                 beta, workspace.data_ptr(), workspace.numel(),
                                                 _stream_ptr(A))
    if st != 0:
        raise ZiplmError(st, "ziplm_hessian_accumulate_tokens")
    return H


def damped_inverse(H: torch.Tensor, damp_frac: float, workspace: Optional[torch.Tensor] = None):
    """(Hinv [L, d, d] float64, layer_status [L] int32) for H [L, d, d] fp32."""
    lib = load_library()
    _check(H, torch.float32, "H")
    L, d, _ = H.shape
    Hinv = torch.empty(L, d, d, dtype=torch.float64, device=H.device)
    status = torch.zeros(L, dtype=torch.int32, device=H.device)
    if workspace is None:
        workspace = _workspace(inverse_workspace_bytes(L, d), H.device)
    with torch.cuda.device(H.device):
        st = lib.ziplm_damped_inverse(H.data_ptr(), L, d, damp_frac, Hinv.data_ptr(),
                                      status.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                      _stream_ptr(H))
    if st != 0:
        raise ZiplmError(st, "ziplm_damped_inverse")
    return Hinv, status


def damped_inverse_noalloc(H: torch.Tensor, damp_frac: float, Hinv: torch.Tensor,
                           layer_status: torch.Tensor) -> None:
    """ziplm_damped_inverse_noalloc: the damped inverse for callers that must not allocate.

    The scratch comes from a 12 MiB array inside the library, so this wrapper allocates nothing
    either: the caller passes the input H [L, d, d] fp32 and both outputs, Hinv [L, d, d]
    float64 and layer_status [L] int32.  Requests with inverse_workspace_bytes(L, d) > 12 MiB
    raise ZiplmError(ERR_UNSUPPORTED).  Calls that overlap on the GPU race on the shared scratch.
    """
    lib = load_library()
    _check(H, torch.float32, "H")
    _check(Hinv, torch.float64, "Hinv")
    _check(layer_status, torch.int32, "layer_status")
    L, d, _ = H.shape
    if tuple(Hinv.shape) != (L, d, d) or layer_status.numel() != L:
        raise ValueError("Hinv must be [L, d, d] and layer_status [L]")
    with torch.cuda.device(H.device):
        st = lib.ziplm_damped_inverse_noalloc(H.data_ptr(), L, d, damp_frac, Hinv.data_ptr(),
                                              layer_status.data_ptr(), _stream_ptr(H))
    if st != 0:
        raise ZiplmError(st, "ziplm_damped_inverse_noalloc")


def prune_layers(W: torch.Tensor, H: torch.Tensor, group_size: int, damp_frac: float,
                 levels: Sequence[int], want_base_loss: bool = True, want_saliency: bool = True,
                 workspace: Optional[torch.Tensor] = None, out: Optional[dict] = None) -> dict:
    """Greedy structured pruning of L same-shape layers; see ziplm_prune_layers in ziplm.h.

    Returns a dict of CUDA tensors: W_snap [L, n_levels, r, d], loss [L, n_levels], base_loss [L]
    (or None), order [L, G] int32, saliency [L, G] (or None), layer_status [L] int32, and the
    workspace that was used.  Pass ``out`` (a dict from an earlier call) to reuse its buffers,
    the workspace included when it is large enough and none is given.
    """
    lib = load_library()
    _check(W, torch.float32, "W")
    _check(H, torch.float32, "H")
    L, r, d = W.shape
    if tuple(H.shape) != (L, d, d):
        raise ValueError("H must be [L, d_col, d_col]")
    levels = [int(v) for v in levels]
    n_levels = len(levels)
    G = d // group_size if group_size > 0 and d % group_size == 0 else 0
    dev = W.device
    if out is None:
        out = dict(
            W_snap=torch.empty(L, n_levels, r, d, dtype=torch.float32, device=dev),
            loss=torch.empty(L, n_levels, dtype=torch.float32, device=dev),
            base_loss=torch.empty(L, dtype=torch.float32, device=dev) if want_base_loss else None,
            order=torch.empty(L, max(G, 1), dtype=torch.int32, device=dev),
            saliency=torch.empty(L, max(G, 1), dtype=torch.float32, device=dev) if want_saliency else None,
            layer_status=torch.empty(L, dtype=torch.int32, device=dev),
        )
    if workspace is None:
        need = prune_workspace_bytes(L, r, d, group_size, n_levels)
        kept = out.get("workspace")          # the workspace of the call that produced ``out``
        if kept is not None and kept.device == dev and kept.numel() >= need:
            workspace = kept
        else:
            out["workspace"] = None          # let go of it before a new one is allocated
            workspace = _workspace(need, dev)
    lv = (ctypes.c_int * max(n_levels, 1))(*levels)
    with torch.cuda.device(dev):
        st = lib.ziplm_prune_layers(W.data_ptr(), H.data_ptr(), L, r, d, group_size, damp_frac, lv,
                                    n_levels, _ptr(out["W_snap"]), _ptr(out["loss"]),
                                    _ptr(out["base_loss"]), _ptr(out["order"]), _ptr(out["saliency"]),
                                    _ptr(out["layer_status"]), workspace.data_ptr(),
                                    workspace.numel(), _stream_ptr(W))
    if st != 0:
        raise ZiplmError(st, "ziplm_prune_layers")
    out["workspace"] = workspace
    return out


def kept_structures(order: torch.Tensor, level: int):
    """(kept [L, level] int32 ascending, layer_status [L] int32) from the removal order [L, G] of
    prune_layers; see ziplm_kept_structures."""
    lib = load_library()
    _check(order, torch.int32, "order")
    L, G = order.shape
    kept = torch.empty(L, max(level, 0), dtype=torch.int32, device=order.device)
    status = torch.empty(L, dtype=torch.int32, device=order.device)
    with torch.cuda.device(order.device):
        st = lib.ziplm_kept_structures(order.data_ptr(), L, G, level, kept.data_ptr(),
                                       status.data_ptr(), _stream_ptr(order))
    if st != 0:
        raise ZiplmError(st, "ziplm_kept_structures")
    return kept, status


def _strided_layers(M: torch.Tensor, name: str):
    if M.dim() != 3 or not M.is_cuda or M.dtype != torch.float32 or (M.shape[2] > 1 and M.stride(2) != 1):
        raise ValueError(f"{name} must be a CUDA fp32 tensor [L, rows, cols] with contiguous rows")
    return M.stride(1) if M.shape[1] > 1 else M.shape[2], M.stride(0) if M.shape[0] > 1 else 0


def gather_columns(M: torch.Tensor, kept: torch.Tensor, group_size: int) -> torch.Tensor:
    """out[l, i, k*g + c] = M[l, i, kept[l, k]*g + c]; M [L, rows, G*g] fp32 (may be a strided view,
    e.g. ``W_snap[:, slot]``); see ziplm_gather_columns."""
    lib = load_library()
    ld, ls = _strided_layers(M, "M")
    _check(kept, torch.int32, "kept")
    L, rows, width = M.shape
    level = kept.shape[1]
    G = width // group_size
    out = torch.empty(L, rows, level * group_size, dtype=torch.float32, device=M.device)
    with torch.cuda.device(M.device):
        st = lib.ziplm_gather_columns(M.data_ptr(), ld, ls, kept.data_ptr(), L, rows, G, group_size,
                                      level, out.data_ptr(), _stream_ptr(M))
    if st != 0:
        raise ZiplmError(st, "ziplm_gather_columns")
    return out


def gather_rows(M: torch.Tensor, kept: torch.Tensor, group_size: int) -> torch.Tensor:
    """out[l, k*g + c, :] = M[l, kept[l, k]*g + c, :]; M [L, G*g, cols] fp32; see
    ziplm_gather_rows."""
    lib = load_library()
    ld, ls = _strided_layers(M, "M")
    _check(kept, torch.int32, "kept")
    L, height, cols = M.shape
    level = kept.shape[1]
    G = height // group_size
    out = torch.empty(L, level * group_size, cols, dtype=torch.float32, device=M.device)
    with torch.cuda.device(M.device):
        st = lib.ziplm_gather_rows(M.data_ptr(), ld, ls, kept.data_ptr(), L, cols, G, group_size,
                                   level, out.data_ptr(), _stream_ptr(M))
    if st != 0:
        raise ZiplmError(st, "ziplm_gather_rows")
    return out


def select_workspace_bytes(n_candidates: int, n_modules: int, n_buckets: int) -> int:
    return int(load_library().ziplm_select_workspace_bytes(n_candidates, n_modules, n_buckets))


def select_levels(loss: torch.Tensor, base_loss: torch.Tensor, time: torch.Tensor,
                  n_options: torch.Tensor, coef: torch.Tensor, budget: float, n_buckets: int,
                  workspace: Optional[torch.Tensor] = None) -> dict:
    """One database level per module under a run-time budget, for every row of ``coef``
    [n_candidates, n_modules]; see ziplm_select_levels.  Returns CUDA tensors selected
    [n_candidates, n_modules] int32, cost and time_sum [n_candidates] float64, status int32."""
    lib = load_library()
    _check(loss, torch.float32, "loss")
    _check(time, torch.float32, "time")
    _check(base_loss, torch.float32, "base_loss")
    _check(n_options, torch.int32, "n_options")
    _check(coef, torch.float32, "coef")
    n_mod, max_opt = loss.shape
    K = coef.shape[0]
    if tuple(time.shape) != (n_mod, max_opt) or base_loss.numel() != n_mod or \
            n_options.numel() != n_mod or coef.shape[1] != n_mod:
        raise ValueError("shapes: loss/time [n_modules, max_options], base_loss/n_options [n_modules], "
                         "coef [n_candidates, n_modules]")
    dev = loss.device
    out = dict(selected=torch.empty(K, n_mod, dtype=torch.int32, device=dev),
               cost=torch.empty(K, dtype=torch.float64, device=dev),
               time_sum=torch.empty(K, dtype=torch.float64, device=dev),
               status=torch.empty(K, dtype=torch.int32, device=dev))
    if workspace is None:
        workspace = _workspace(select_workspace_bytes(K, n_mod, n_buckets), dev)
    with torch.cuda.device(dev):
        st = lib.ziplm_select_levels(loss.data_ptr(), base_loss.data_ptr(), time.data_ptr(),
                                     n_options.data_ptr(), n_mod, max_opt, coef.data_ptr(), K,
                                     float(budget), n_buckets, out["selected"].data_ptr(),
                                     out["cost"].data_ptr(), out["time_sum"].data_ptr(),
                                     out["status"].data_ptr(), workspace.data_ptr(), workspace.numel(),
                                     _stream_ptr(loss))
    if st != 0:
        raise ZiplmError(st, "ziplm_select_levels")
    return out


def search_workspace_bytes(n_searches: int, n_modules: int, n_buckets: int) -> int:
    return int(load_library().ziplm_search_workspace_bytes(n_searches, n_modules, n_buckets))


def search_levels(loss: torch.Tensor, base_loss: torch.Tensor, time: torch.Tensor,
                  n_options: torch.Tensor, objective: torch.Tensor, coef0: torch.Tensor,
                  budgets: torch.Tensor, n_buckets: int, mask: torch.Tensor, values: torch.Tensor,
                  workspace: Optional[torch.Tensor] = None) -> dict:
    """Mutation search over the sensitivity coefficients, one search per budget; see
    ziplm_search_levels.  mask [S, n_steps, n_modules] uint8, values the same shape fp32."""
    lib = load_library()
    for t, dt, name in ((loss, torch.float32, "loss"), (time, torch.float32, "time"),
                        (base_loss, torch.float32, "base_loss"), (n_options, torch.int32, "n_options"),
                        (objective, torch.float32, "objective"), (coef0, torch.float32, "coef0"),
                        (budgets, torch.float64, "budgets"), (mask, torch.uint8, "mask"),
                        (values, torch.float32, "values")):
        _check(t, dt, name)
    n_mod, max_opt = loss.shape
    S, n_steps = mask.shape[0], mask.shape[1]
    if tuple(mask.shape) != (S, n_steps, n_mod) or tuple(values.shape) != (S, n_steps, n_mod) or \
            tuple(coef0.shape) != (S, n_mod) or budgets.numel() != S or \
            tuple(objective.shape) != (n_mod, max_opt) or tuple(time.shape) != (n_mod, max_opt):
        raise ValueError("shapes: mask/values [S, n_steps, n_modules], coef0 [S, n_modules], budgets [S]")
    dev = loss.device
    out = dict(selected=torch.empty(S, n_mod, dtype=torch.int32, device=dev),
               coef=torch.empty(S, n_mod, dtype=torch.float32, device=dev),
               objective=torch.empty(S, dtype=torch.float64, device=dev),
               n_accepted=torch.empty(S, dtype=torch.int32, device=dev),
               status=torch.empty(S, dtype=torch.int32, device=dev))
    if workspace is None:
        workspace = _workspace(search_workspace_bytes(S, n_mod, n_buckets), dev)
    with torch.cuda.device(dev):
        st = lib.ziplm_search_levels(loss.data_ptr(), base_loss.data_ptr(), time.data_ptr(),
                                     n_options.data_ptr(), n_mod, max_opt, objective.data_ptr(),
                                     coef0.data_ptr(), budgets.data_ptr(), S, n_buckets,
                                     mask.data_ptr(), values.data_ptr(), n_steps,
                                     out["selected"].data_ptr(), out["coef"].data_ptr(),
                                     out["objective"].data_ptr(), out["n_accepted"].data_ptr(),
                                     out["status"].data_ptr(), workspace.data_ptr(), workspace.numel(),
                                     _stream_ptr(loss))
    if st != 0:
        raise ZiplmError(st, "ziplm_search_levels")
    return out


class Option:
    """Diagnostic options of ziplm_set_option (all default to 0)."""
    NEURON_PATH = 0          # 1: per-step streaming update instead of delayed rank-32 updates
    LAYER_GROUPS = 1         # 1..8 layer groups on internal streams (0: default)
    FORCE_BLOCK_PATH = 2     # 1: group_size 1 through the general block path
    HESSIAN_ROUTE = 3        # 1: CUDA-core Hessian kernel always
    SPIN_LIMIT = 4           # poll limit of the Hessian kernel's wait for a free pipeline stage
    COMPACT_EVERY_BLOCK = 5  # 1: squeeze removed positions out after every block of the neuron path


def set_option(option: int, value: int) -> None:
    st = load_library().ziplm_set_option(int(option), int(value))
    if st != 0:
        raise ZiplmError(st, "ziplm_set_option")


def get_option(option: int) -> int:
    return int(load_library().ziplm_get_option(int(option)))


def launch_count() -> int:
    """Kernels launched by the library since it was loaded."""
    return int(load_library().ziplm_launch_count())


def profile_begin() -> None:
    """Switch on per-phase CUDA-event timing for the calls that follow."""
    st = load_library().ziplm_profile_begin()
    if st != 0:
        raise ZiplmError(st, "ziplm_profile_begin")


def profile_end() -> dict:
    """Switch timing off and return {phase name: (milliseconds, spans)} (synchronises)."""
    lib = load_library()
    n = lib.ziplm_profile_phase_count()
    ms = (ctypes.c_double * n)()
    cnt = (ctypes.c_longlong * n)()
    st = lib.ziplm_profile_end(ms, cnt, n)
    if st != 0:
        raise ZiplmError(st, "ziplm_profile_end")
    return {lib.ziplm_profile_phase_name(i).decode(): (ms[i], int(cnt[i])) for i in range(n)}


def profile_phase_count() -> int:
    return int(load_library().ziplm_profile_phase_count())


def profile_phase_name(i: int) -> str:
    return load_library().ziplm_profile_phase_name(i).decode()
