"""ctypes binding of liblt_indexer.so: same names as the C ABI, argument marshalling only.

Every function takes torch CUDA tensors (used purely as device memory), passes
their pointers and sizes to the library and returns.  No arithmetic of the
method happens here, and there is no fallback: if the library is missing the
first call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

LT_DTYPE_F32, LT_DTYPE_BF16, LT_DTYPE_E4M3 = 0, 1, 2
LT_PATH_AUTO, LT_PATH_FUSED, LT_PATH_GENERIC, LT_PATH_FUSED_ABS = 0, 1, 2, 3
LT_OK = 0
LT_STATUS_TIMEOUT, LT_STATUS_FALLBACK, LT_STATUS_BOUNDS = 1, 2, 4
LT_DEBUG_SKIP_ONE_KTILE = 1
LT_MAX_TOPK = 8192

_DTYPE_CODES = {"f32": LT_DTYPE_F32, "bf16": LT_DTYPE_BF16, "e4m3": LT_DTYPE_E4M3}


class LtError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what} failed: {code} ({strerror(code)})")
        self.code = code


class Tunables(ctypes.Structure):
    """Mirror of `lt_tunables`; zero fields mean "default"."""

    _fields_ = [("path", ctypes.c_int), ("cap_mult", ctypes.c_int), ("sample_mult", ctypes.c_int),
                ("segment_tiles", ctypes.c_int), ("grid", ctypes.c_int), ("sample_rank", ctypes.c_int),
                ("wait_limit_us", ctypes.c_int), ("debug_flags", ctypes.c_int)]


_lib = None
_lib_path = None


def library_path() -> str:
    """The build `load()` opens: `use_library()`'s choice, else $LT_INDEXER_LIB, else the in-tree release build."""
    return _lib_path or os.environ.get("LT_INDEXER_LIB") or _build.LIB_PATH


def use_library(path: Optional[str]) -> None:
    """Selects which build of the library `load()` opens (None: the release build).  Used by the tests
    that run the bounds-checking build (`build.build(debug_bounds=True)`)."""
    global _lib, _lib_path
    _lib_path = path
    _lib = None


def load() -> ctypes.CDLL:
    """Loads the shared library (built in-tree by `build.build()`); raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: run `python -m paper_2607_11976_b200.build` (needs nvcc); "
                           "there is no CPU or PyTorch fallback for this path")
    lib = ctypes.CDLL(path)
    vp, fp, ip, i, sz = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    lib.lt_indexer_topk.argtypes = [vp, fp, vp, fp, i, i, i, i, i, i, ip, fp, vp]
    lib.lt_indexer_topk.restype = i
    lib.lt_indexer_topk_ex.argtypes = [i, vp, fp, vp, fp, i, i, i, i, i, i, ip, fp, vp, sz, ctypes.POINTER(Tunables), vp]
    lib.lt_indexer_topk_ex.restype = i
    lib.lt_indexer_topk_workspace_bytes.argtypes = [i, i, i, i, i, i, ctypes.POINTER(Tunables)]
    lib.lt_indexer_topk_workspace_bytes.restype = sz
    lib.lt_indexer_topk_sampled.argtypes = [i, vp, fp, vp, fp, i, i, i, i, i, i, ip, i, ip, fp, vp, sz, ctypes.POINTER(Tunables), vp]
    lib.lt_indexer_topk_sampled.restype = i
    lib.lt_indexer_topk_sampled_workspace_bytes.argtypes = [i, i, i, i, i, i, i, ctypes.POINTER(Tunables)]
    lib.lt_indexer_topk_sampled_workspace_bytes.restype = sz
    lib.lt_indexer_topk_paged.argtypes = [i, vp, fp, vp, fp, ip, i, ctypes.c_longlong, i, i, i, i, i, i, ip, fp, vp, sz,
                                          ctypes.POINTER(Tunables), vp]
    lib.lt_indexer_topk_paged.restype = i
    lib.lt_indexer_topk_paged_workspace_bytes.argtypes = [i, i, i, i, i, i, ctypes.POINTER(Tunables)]
    lib.lt_indexer_topk_paged_workspace_bytes.restype = sz
    lib.lt_topk_frequent.argtypes = [ip, i, i, i, i, ip, ip, vp, sz, vp]
    lib.lt_topk_frequent.restype = i
    lib.lt_topk_frequent_workspace_bytes.argtypes = [i]
    lib.lt_topk_frequent_workspace_bytes.restype = sz
    lib.lt_knn_topk.argtypes = [i, vp, vp, i, i, i, i, ip, fp, vp, sz, ctypes.POINTER(Tunables), vp]
    lib.lt_knn_topk.restype = i
    lib.lt_knn_topk_workspace_bytes.argtypes = [i, i, i, i, i, ctypes.POINTER(Tunables)]
    lib.lt_knn_topk_workspace_bytes.restype = sz
    lib.lt_knn_scores.argtypes = [i, vp, vp, i, i, i, i, i, fp, vp]
    lib.lt_knn_scores.restype = i
    lib.lt_dsa_union_mask.argtypes = [ip, i, i, i, i, ip, ip, vp, vp]
    lib.lt_dsa_union_mask.restype = i
    lib.lt_indexer_sample_plan.argtypes = [i, i, i, ctypes.POINTER(Tunables), ctypes.POINTER(ctypes.c_int)]
    lib.lt_indexer_sample_plan.restype = i
    lib.lt_indexer_scores.argtypes = [i, vp, fp, vp, fp, i, i, i, i, i, i, i, fp, i, vp]
    lib.lt_indexer_scores.restype = i
    lib.lt_unfused_topk.argtypes = [i, vp, fp, vp, fp, i, i, i, i, i, i, ip, fp, fp, sz, i, vp]
    lib.lt_unfused_topk.restype = i
    lib.lt_indexer_topk_static.argtypes = [i, vp, fp, vp, fp, i, i, i, i, i, i, ip, fp, vp]
    lib.lt_indexer_topk_static.restype = i
    lib.lt_read_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int), vp]
    lib.lt_read_status.restype = i
    lib.lt_indexer_topk_static_max_keys.restype = i
    lib.lt_read_status_static.argtypes = [ctypes.POINTER(ctypes.c_int), vp]
    lib.lt_read_status_static.restype = i
    lib.lt_debug_wait_timeout.argtypes = [i, ip, vp]
    lib.lt_debug_wait_timeout.restype = i
    lib.lt_debug_umma_stream.argtypes = [i, i, ip, vp]
    lib.lt_debug_umma_stream.restype = i
    lib.lt_indexer_topk_strided.argtypes = [i, vp, fp, vp, ctypes.c_longlong, fp, i, i, i, i, i, i, ip, fp, vp, sz,
                                            ctypes.POINTER(Tunables), vp]
    lib.lt_indexer_topk_strided.restype = i
    lib.lt_launch_count.restype = ctypes.c_ulonglong
    lib.lt_set_profiling.argtypes = [i]
    lib.lt_set_profiling.restype = i
    lib.lt_read_phase_ms.argtypes = [ctypes.POINTER(ctypes.c_float), vp]
    lib.lt_read_phase_ms.restype = i
    lib.lt_strerror.argtypes = [i]
    lib.lt_strerror.restype = ctypes.c_char_p
    lib.lt_last_cuda_error.restype = i
    lib.lt_version.restype = i
    lib.lt_shutdown.restype = None
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load().lt_strerror(code).decode()


def dtype_code(dtype) -> int:
    return _DTYPE_CODES[dtype] if isinstance(dtype, str) else int(dtype)


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(code: int, what: str) -> None:
    if code != LT_OK:
        extra = f" (cudaError {load().lt_last_cuda_error()})" if code == -4 else ""
        raise LtError(code, what + extra)


def _shape(q: torch.Tensor, k: torch.Tensor):
    T, H, D = q.shape
    N, D2 = k.shape
    if D2 != D:
        raise ValueError("q and k disagree on D")
    return T, N, H, D


def lt_indexer_topk_workspace_bytes(dtype, T: int, N: int, H: int, D: int, topk: int,
                                    tunables: Optional[Tunables] = None) -> int:
    return int(load().lt_indexer_topk_workspace_bytes(dtype_code(dtype), T, N, H, D, topk,
                                                      ctypes.byref(tunables) if tunables else None))


def lt_indexer_sample_plan(N: int, topk: int, causal_offset: int, tunables: Optional[Tunables] = None):
    """(sample size, stride, rank) the fused path uses for this problem; host-only."""
    buf = (ctypes.c_int * 3)()
    _check(load().lt_indexer_sample_plan(N, topk, causal_offset, ctypes.byref(tunables) if tunables else None, buf),
           "lt_indexer_sample_plan")
    return tuple(buf)


def lt_indexer_topk(q, w, k, k_scale, topk: int, causal_offset: int, out_idx, out_score=None, stream=None) -> None:
    """13-argument C entry point: dtype inferred from k_scale (None -> bf16, else e4m3)."""
    T, N, H, D = _shape(q, k)
    _check(load().lt_indexer_topk(_ptr(q), _ptr(w), _ptr(k), _ptr(k_scale), T, N, H, D, topk, causal_offset,
                                  _ptr(out_idx), _ptr(out_score), _stream(stream)), "lt_indexer_topk")


def lt_indexer_topk_ex(dtype, q, w, k, k_scale, topk: int, causal_offset: int, out_idx, out_score, workspace,
                       tunables: Optional[Tunables] = None, stream=None) -> None:
    T, N, H, D = _shape(q, k)
    _check(load().lt_indexer_topk_ex(dtype_code(dtype), _ptr(q), _ptr(w), _ptr(k), _ptr(k_scale), T, N, H, D, topk,
                                     causal_offset, _ptr(out_idx), _ptr(out_score), _ptr(workspace),
                                     workspace.numel() * workspace.element_size(),
                                     ctypes.byref(tunables) if tunables else None, _stream(stream)), "lt_indexer_topk_ex")


def lt_indexer_topk_strided(dtype, q, w, k_view, k_scale, topk: int, causal_offset: int, out_idx, out_score, workspace,
                            tunables: Optional[Tunables] = None, stream=None) -> None:
    """lt_indexer_topk_ex over a row-strided key view: `k_view` is an [N, D] CUDA tensor whose rows are
    `k_view.stride(0)` elements apart (inner stride 1), e.g. `cache[:, :D]` of a wider cache."""
    T, H, D = q.shape
    N, D2 = k_view.shape
    if D2 != D or k_view.stride(1) != 1 or not k_view.is_cuda:
        raise ValueError("expected an [N, D] CUDA view with unit inner stride")
    _check(load().lt_indexer_topk_strided(dtype_code(dtype), _ptr(q), _ptr(w), ctypes.c_void_p(k_view.data_ptr()),
                                          int(k_view.stride(0)), _ptr(k_scale), T, N, H, D, topk, causal_offset,
                                          _ptr(out_idx), _ptr(out_score), _ptr(workspace),
                                          workspace.numel() * workspace.element_size(),
                                          ctypes.byref(tunables) if tunables else None, _stream(stream)),
           "lt_indexer_topk_strided")


def lt_indexer_topk_sampled_workspace_bytes(dtype, T: int, N: int, H: int, D: int, topk: int, n_sample: int,
                                            tunables: Optional[Tunables] = None) -> int:
    return int(load().lt_indexer_topk_sampled_workspace_bytes(dtype_code(dtype), T, N, H, D, topk, n_sample,
                                                              ctypes.byref(tunables) if tunables else None))


def lt_indexer_topk_sampled(dtype, q, w, k, k_scale, topk: int, causal_offset: int, sample_idx, out_idx, out_score, workspace,
                            tunables: Optional[Tunables] = None, stream=None) -> None:
    """lt_indexer_topk_ex with a caller-provided sample (int32 device tensor of key positions)."""
    T, N, H, D = _shape(q, k)
    _check(load().lt_indexer_topk_sampled(dtype_code(dtype), _ptr(q), _ptr(w), _ptr(k), _ptr(k_scale), T, N, H, D, topk,
                                          causal_offset, _ptr(sample_idx), sample_idx.numel(), _ptr(out_idx), _ptr(out_score),
                                          _ptr(workspace), workspace.numel() * workspace.element_size(),
                                          ctypes.byref(tunables) if tunables else None, _stream(stream)),
           "lt_indexer_topk_sampled")


def lt_indexer_topk_paged_workspace_bytes(dtype, T: int, N: int, H: int, D: int, topk: int,
                                          tunables: Optional[Tunables] = None) -> int:
    return int(load().lt_indexer_topk_paged_workspace_bytes(dtype_code(dtype), T, N, H, D, topk,
                                                            ctypes.byref(tunables) if tunables else None))


def lt_indexer_topk_paged(dtype, q, w, k_pool, k_scale_pool, page_table, N: int, topk: int, causal_offset: int, out_idx,
                          out_score, workspace, tunables: Optional[Tunables] = None, stream=None) -> None:
    """lt_indexer_topk_ex over a paged key cache: k_pool [pool_rows, D], page_table int32 [n_pages] (pages of 64 keys)."""
    T, H, D = q.shape
    pool_rows, D2 = k_pool.shape
    if D2 != D:
        raise ValueError("q and k_pool disagree on D")
    _check(load().lt_indexer_topk_paged(dtype_code(dtype), _ptr(q), _ptr(w), _ptr(k_pool), _ptr(k_scale_pool), _ptr(page_table),
                                        page_table.numel(), pool_rows, T, N, H, D, topk, causal_offset, _ptr(out_idx),
                                        _ptr(out_score), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                        ctypes.byref(tunables) if tunables else None, _stream(stream)), "lt_indexer_topk_paged")


def lt_topk_frequent_workspace_bytes(N: int) -> int:
    return int(load().lt_topk_frequent_workspace_bytes(N))


def lt_topk_frequent(idx, N: int, out_pos, out_count, workspace, stream=None) -> None:
    """out_pos (int32 device tensor of n_out elements) = the most frequent positions of the [T, topk] matrix idx."""
    T, topk = idx.shape
    _check(load().lt_topk_frequent(_ptr(idx), T, topk, N, out_pos.numel(), _ptr(out_pos), _ptr(out_count), _ptr(workspace),
                                   workspace.numel() * workspace.element_size(), _stream(stream)), "lt_topk_frequent")


def lt_knn_topk_workspace_bytes(T: int, N: int, D: int, topk: int, tunables: Optional[Tunables] = None) -> int:
    return int(load().lt_knn_topk_workspace_bytes(LT_DTYPE_BF16, T, N, D, topk, ctypes.byref(tunables) if tunables else None))


def lt_knn_topk(q, x, topk: int, out_idx, out_score, workspace, tunables: Optional[Tunables] = None, stream=None) -> None:
    """Exact top-k inner products of the bf16 queries q [T, D] over the bf16 corpus x [N, D]."""
    T, D = q.shape
    N, D2 = x.shape
    if D2 != D:
        raise ValueError("q and x disagree on D")
    _check(load().lt_knn_topk(LT_DTYPE_BF16, _ptr(q), _ptr(x), T, N, D, topk, _ptr(out_idx), _ptr(out_score), _ptr(workspace),
                              workspace.numel() * workspace.element_size(), ctypes.byref(tunables) if tunables else None,
                              _stream(stream)), "lt_knn_topk")


def lt_knn_scores(q, x, row_begin: int, row_end: int, out_scores, stream=None) -> None:
    T, D = q.shape
    N = x.shape[0]
    _check(load().lt_knn_scores(LT_DTYPE_BF16, _ptr(q), _ptr(x), T, N, D, row_begin, row_end, _ptr(out_scores), _stream(stream)),
           "lt_knn_scores")


def lt_dsa_union_mask(idx, N: int, group: int, union_pos, union_len, member_mask, stream=None) -> None:
    """LiteDSA union list + membership masks of consecutive groups of `group` rows of the [T, topk] matrix idx."""
    T, topk = idx.shape
    _check(load().lt_dsa_union_mask(_ptr(idx), T, topk, N, group, _ptr(union_pos), _ptr(union_len), _ptr(member_mask),
                                    _stream(stream)), "lt_dsa_union_mask")


def lt_indexer_scores(dtype, q, w, k, k_scale, causal_offset: int, row_begin: int, row_end: int, out_scores,
                      path: int = LT_PATH_AUTO, stream=None) -> None:
    T, N, H, D = _shape(q, k)
    _check(load().lt_indexer_scores(dtype_code(dtype), _ptr(q), _ptr(w), _ptr(k), _ptr(k_scale), T, N, H, D, causal_offset,
                                    row_begin, row_end, _ptr(out_scores), path, _stream(stream)), "lt_indexer_scores")


def lt_unfused_topk(dtype, q, w, k, k_scale, topk: int, causal_offset: int, out_idx, out_score, score_buf,
                    path: int = LT_PATH_AUTO, stream=None) -> None:
    T, N, H, D = _shape(q, k)
    _check(load().lt_unfused_topk(dtype_code(dtype), _ptr(q), _ptr(w), _ptr(k), _ptr(k_scale), T, N, H, D, topk,
                                  causal_offset, _ptr(out_idx), _ptr(out_score), _ptr(score_buf),
                                  score_buf.numel() * score_buf.element_size(), path, _stream(stream)), "lt_unfused_topk")


def lt_indexer_topk_static(dtype, q, w, k, k_scale, topk: int, causal_offset: int, out_idx, out_score=None, stream=None) -> None:
    """Allocation-free entry point: same result as lt_indexer_topk_ex, scratch inside the library
    (16 MiB per GPU, one score row must fit: N <= 4,194,240).  Calls that may overlap on the GPU race."""
    T, N, H, D = _shape(q, k)
    _check(load().lt_indexer_topk_static(dtype_code(dtype), _ptr(q), _ptr(w), _ptr(k), _ptr(k_scale), T, N, H, D, topk,
                                         causal_offset, _ptr(out_idx), _ptr(out_score), _stream(stream)),
           "lt_indexer_topk_static")


def lt_read_status(workspace=None, stream=None) -> list:
    """Synchronises the stream and returns the 8-int status block of a workspace
    (None: the library-owned workspace of lt_indexer_topk)."""
    buf = (ctypes.c_int * 8)()
    _check(load().lt_read_status(_ptr(workspace), buf, _stream(stream)), "lt_read_status")
    return list(buf)


def lt_read_status_static(stream=None) -> list:
    """The status block of the last lt_indexer_topk_static call on the current device."""
    buf = (ctypes.c_int * 8)()
    _check(load().lt_read_status_static(buf, _stream(stream)), "lt_read_status_static")
    return list(buf)


def lt_debug_wait_timeout(limit_us: int, result2, stream=None) -> None:
    """Runs the bounded-wait probe: result2 (int32 CUDA tensor of 2) receives (wait result, abort flag)."""
    _check(load().lt_debug_wait_timeout(int(limit_us), _ptr(result2), _stream(stream)), "lt_debug_wait_timeout")


def lt_debug_umma_stream(pair: bool, iters: int, status, stream=None) -> None:
    """Enqueues one launch of the bare FP8 UMMA stream; status: zeroed int32 CUDA tensor of 1."""
    _check(load().lt_debug_umma_stream(1 if pair else 0, int(iters), _ptr(status), _stream(stream)), "lt_debug_umma_stream")


def lt_launch_count() -> int:
    return int(load().lt_launch_count())


def lt_set_profiling(enable: bool) -> None:
    _check(load().lt_set_profiling(1 if enable else 0), "lt_set_profiling")


def lt_read_phase_ms(stream=None) -> list:
    """Device ms of [sample scoring, sample statistics, fused scan, final select, fallback]."""
    buf = (ctypes.c_float * 5)()
    _check(load().lt_read_phase_ms(buf, _stream(stream)), "lt_read_phase_ms")
    return list(buf)


# ---------------------------------------------------------------------------------------------
# device-memory helpers (plumbing only)
# ---------------------------------------------------------------------------------------------

def to_device(inp, device="cuda"):
    """Uploads a workload (numpy storage codes) as torch tensors: (q, w, k, k_scale)."""
    def up(a):
        return None if a is None else torch.from_numpy(a).to(device)

    if inp.dtype == "bf16":
        q = torch.from_numpy(inp.q.view("int16")).to(device).view(torch.bfloat16)
        k = torch.from_numpy(inp.k.view("int16")).to(device).view(torch.bfloat16)
    else:
        q, k = up(inp.q), up(inp.k)
    return q, up(inp.w), k, up(inp.k_scale)


def alloc_workspace(dtype, T, N, H, D, topk, tunables: Optional[Tunables] = None, device="cuda") -> torch.Tensor:
    nbytes = lt_indexer_topk_workspace_bytes(dtype, T, N, H, D, topk, tunables)
    if nbytes == 0:
        raise ValueError("invalid problem for lt_indexer_topk_workspace_bytes")
    return torch.empty(nbytes, dtype=torch.uint8, device=device)
