"""ctypes binding of libdapq.so: argument marshalling only.

Every function has the name and the argument order of its C entry point in
include/dapq.h; torch tensors are passed as raw device (or host) pointers and the
current torch CUDA stream is used unless one is given.  Nothing is computed here.
The library must have been built (python -m paper_2603_11564_b200.build); there is
no fallback: a missing library raises ImportError at first use.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libdapq.so")

DAPQ_OK, DAPQ_ERR_INVALID_ARG, DAPQ_ERR_UNSUPPORTED, DAPQ_ERR_WORKSPACE, DAPQ_ERR_CUDA, \
    DAPQ_ERR_TIMEOUT = range(6)
DAPQ_BF16, DAPQ_F32 = 0, 1
DAPQ_POOL_NONE, DAPQ_POOL_MAX, DAPQ_POOL_AVG = 0, 1, 2
DAPQ_FLAG_CUDA_CORE_SCORER = 1
DAPQ_FLAG_ROPE_INTERLEAVED = 2
DAPQ_FLAG_Q_BF16, DAPQ_FLAG_Q_LO_SWEEP1, DAPQ_FLAG_Q_LO_SWEEP2 = 4, 8, 16
_STATUS_NAMES = {0: "DAPQ_OK", 1: "DAPQ_ERR_INVALID_ARG", 2: "DAPQ_ERR_UNSUPPORTED",
                 3: "DAPQ_ERR_WORKSPACE", 4: "DAPQ_ERR_CUDA", 5: "DAPQ_ERR_TIMEOUT"}

EXPORTS = ("dapq_create", "dapq_destroy", "dapq_last_error", "dapq_poll_status",
           "dapq_launch_count", "dapq_set_wait_limit", "dapq_rope_inv_freq_llama3", "dapq_profile", "dapq_profile_read", "dapq_rope_pseudo_q", "dapq_score", "dapq_topk_select",
           "dapq_compact_kv", "dapq_evict", "dapq_evict_layers", "dapq_evict_host", "dapq_evict_layers_host", "dapq_score_static", "dapq_recall")


class DapqError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{_STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class dapq_shape(C.Structure):
    _fields_ = [("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("n_pseudo", C.c_int32), ("max_batch", C.c_int32), ("dtype", C.c_int32),
                ("max_total_rows", C.c_int64), ("rope_base", C.c_double),
                ("inv_freq_host", C.POINTER(C.c_double)), ("softmax_scale", C.c_float),
                ("pool_mode", C.c_int32), ("pool_kernel", C.c_int32), ("flags", C.c_int32)]


class dapq_cache_view(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p),
                ("k_head_stride", C.c_int64), ("k_row_stride", C.c_int64),
                ("v_head_stride", C.c_int64), ("v_row_stride", C.c_int64),
                ("cu_rows_host", C.POINTER(C.c_int32)), ("prompt_len_host", C.POINTER(C.c_int32)),
                ("batch", C.c_int32), ("reserved", C.c_int32)]


_lib = None


def load_library() -> C.CDLL:
    """dlopen libdapq.so and declare its prototypes (fails loudly if it is missing)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} not found: build it with `python -m paper_2603_11564_b200.build`")
    lib = C.CDLL(_LIB_PATH)
    vp, i32p, f32p = C.c_void_p, C.POINTER(C.c_int32), C.c_void_p
    lib.dapq_create.argtypes = [C.POINTER(vp), C.POINTER(dapq_shape), C.c_int]
    lib.dapq_create.restype = C.c_int
    lib.dapq_destroy.argtypes = [vp]
    lib.dapq_destroy.restype = None
    lib.dapq_last_error.argtypes = [vp]
    lib.dapq_last_error.restype = C.c_char_p
    lib.dapq_poll_status.argtypes = [vp, vp]
    lib.dapq_poll_status.restype = C.c_int
    lib.dapq_launch_count.argtypes = [vp]
    lib.dapq_launch_count.restype = C.c_int64
    lib.dapq_rope_inv_freq_llama3.argtypes = [C.c_double, C.c_double, C.c_double, C.c_double, C.c_int32, C.POINTER(C.c_double)]
    lib.dapq_rope_inv_freq_llama3.restype = C.c_int
    lib.dapq_set_wait_limit.argtypes = [vp, C.c_int64]
    lib.dapq_set_wait_limit.restype = C.c_int
    lib.dapq_profile.argtypes = [vp, C.c_int32]
    lib.dapq_profile.restype = C.c_int
    lib.dapq_profile_read.argtypes = [vp, vp, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    lib.dapq_profile_read.restype = C.c_int
    lib.dapq_rope_pseudo_q.argtypes = [vp, vp, i32p, C.c_int32, vp, vp]
    lib.dapq_rope_pseudo_q.restype = C.c_int
    lib.dapq_score.argtypes = [vp, vp, C.POINTER(dapq_cache_view), f32p, f32p, f32p, f32p, vp]
    lib.dapq_score.restype = C.c_int
    lib.dapq_topk_select.argtypes = [vp, f32p, i32p, i32p, C.c_int32, vp, vp]
    lib.dapq_topk_select.restype = C.c_int
    lib.dapq_compact_kv.argtypes = [vp, C.POINTER(dapq_cache_view), vp, i32p, vp, vp, vp]
    lib.dapq_compact_kv.restype = C.c_int
    lib.dapq_evict.argtypes = [vp, vp, C.POINTER(dapq_cache_view), i32p, vp, vp, vp, f32p, vp]
    lib.dapq_evict.restype = C.c_int
    lib.dapq_evict_layers.argtypes = [vp, C.c_int32, C.POINTER(vp), C.POINTER(dapq_cache_view), i32p, C.c_int64,
                                      C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), vp]
    lib.dapq_evict_layers.restype = C.c_int
    lib.dapq_evict_layers_host.argtypes = lib.dapq_evict_layers.argtypes
    lib.dapq_evict_layers_host.restype = C.c_int
    lib.dapq_evict_host.argtypes = [vp, vp, C.POINTER(dapq_cache_view), i32p, vp, vp, vp, vp]
    lib.dapq_evict_host.restype = C.c_int
    lib.dapq_recall.argtypes = [vp, vp, vp, i32p, i32p, C.c_int32, f32p, vp]
    lib.dapq_recall.restype = C.c_int
    lib.dapq_score_static.argtypes = [C.POINTER(dapq_shape), C.c_int, vp, C.POINTER(dapq_cache_view), f32p, vp,
                                      C.c_char_p, C.c_size_t]
    lib.dapq_score_static.restype = C.c_int
    _lib = lib
    return lib


def _i32(seq: Sequence[int]):
    arr = np.ascontiguousarray(np.asarray(seq, dtype=np.int32))
    return arr, arr.ctypes.data_as(C.POINTER(C.c_int32))


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    return getattr(stream, "cuda_stream", stream) or None


def _check(ctx, st: int) -> None:
    if st != DAPQ_OK:
        raise DapqError(st, load_library().dapq_last_error(ctx).decode())


def _view(k: torch.Tensor, v: Optional[torch.Tensor], cu_rows, prompt_len):
    """dapq_cache_view of [H_kv, R, d] tensors (any head / row strides, d contiguous)."""
    assert k.dim() == 3 and k.stride(2) == 1
    cu, cu_p = _i32(cu_rows)
    pl, pl_p = _i32(prompt_len)
    view = dapq_cache_view()
    view.k = k.data_ptr()
    view.k_head_stride, view.k_row_stride = k.stride(0), k.stride(1)
    if v is not None:
        assert v.dim() == 3 and v.stride(2) == 1
        view.v = v.data_ptr()
        view.v_head_stride, view.v_row_stride = v.stride(0), v.stride(1)
    view.cu_rows_host, view.prompt_len_host = cu_p, pl_p
    view.batch = len(pl)
    view._keep = (cu, pl, k, v)
    return view


def dapq_create(n_q_heads: int, n_kv_heads: int, n_pseudo: int, max_batch: int, max_total_rows: int,
                dtype: int, rope_base: float, head_dim: int = 128, softmax_scale: float = 0.0,
                inv_freq: Optional[Sequence[float]] = None, pool_mode: int = DAPQ_POOL_NONE,
                pool_kernel: int = 1, flags: int = 0, device: int = 0):
    lib = load_library()
    sh = dapq_shape(n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, head_dim=head_dim, n_pseudo=n_pseudo,
                    max_batch=max_batch, dtype=dtype, max_total_rows=max_total_rows,
                    rope_base=rope_base, softmax_scale=softmax_scale, pool_mode=pool_mode,
                    pool_kernel=pool_kernel, flags=flags)
    if inv_freq is not None:
        arr = (C.c_double * len(inv_freq))(*[float(x) for x in inv_freq])
        sh.inv_freq_host = C.cast(arr, C.POINTER(C.c_double))
    ctx = C.c_void_p()
    st = lib.dapq_create(C.byref(ctx), C.byref(sh), device)
    if st != DAPQ_OK:
        raise DapqError(st, lib.dapq_last_error(None).decode())
    return ctx


def dapq_destroy(ctx) -> None:
    load_library().dapq_destroy(ctx)


def dapq_last_error(ctx) -> str:
    return load_library().dapq_last_error(ctx).decode()


def dapq_poll_status(ctx, stream=None) -> None:
    _check(ctx, load_library().dapq_poll_status(ctx, _stream(stream)))


def dapq_launch_count(ctx) -> int:
    return int(load_library().dapq_launch_count(ctx))


PROF_KINDS = ("rope", "sweep1", "lse_merge", "sweep2", "topk", "compact", "pool", "recall", "slot_sum")


def dapq_rope_inv_freq_llama3(rope_base: float = 5.0e5, factor: float = 8.0, low_freq_factor: float = 1.0,
                              high_freq_factor: float = 4.0, original_context: int = 8192):
    """[64] float64 frequencies for dapq_create(inv_freq=...)."""
    out = (C.c_double * 64)()
    st = load_library().dapq_rope_inv_freq_llama3(rope_base, factor, low_freq_factor, high_freq_factor, original_context, out)
    if st != DAPQ_OK:
        raise DapqError(st, "dapq_rope_inv_freq_llama3: bad argument")
    return [float(x) for x in out]


def dapq_set_wait_limit(ctx, cycles: int) -> None:
    _check(ctx, load_library().dapq_set_wait_limit(ctx, int(cycles)))


def dapq_profile(ctx, enable: bool) -> None:
    _check(ctx, load_library().dapq_profile(ctx, 1 if enable else 0))


def dapq_profile_read(ctx, stream=None):
    """{kind: (total_ms, launches)} since profiling was enabled."""
    ms = (C.c_double * len(PROF_KINDS))()
    cnt = (C.c_int64 * len(PROF_KINDS))()
    _check(ctx, load_library().dapq_profile_read(ctx, _stream(stream), ms, cnt))
    return {k: (float(ms[i]), int(cnt[i])) for i, k in enumerate(PROF_KINDS)}


def dapq_rope_pseudo_q(ctx, q_pre: torch.Tensor, pos_start: Sequence[int], q_rot: torch.Tensor,
                       stream=None) -> None:
    assert q_pre.is_contiguous() and q_rot.is_contiguous()
    ps, ps_p = _i32(pos_start)
    _check(ctx, load_library().dapq_rope_pseudo_q(ctx, q_pre.data_ptr(), ps_p, len(ps), q_rot.data_ptr(),
                                                  _stream(stream)))


def dapq_score(ctx, q_rot: torch.Tensor, k: torch.Tensor, cu_rows, prompt_len, scores: torch.Tensor,
               lse_in: Optional[torch.Tensor] = None, lse_out: Optional[torch.Tensor] = None,
               syn_mass: Optional[torch.Tensor] = None, stream=None) -> None:
    view = _view(k, None, cu_rows, prompt_len)
    _check(ctx, load_library().dapq_score(ctx, q_rot.data_ptr(), C.byref(view), _ptr(lse_in), scores.data_ptr(),
                                          _ptr(lse_out), _ptr(syn_mass), _stream(stream)))


def dapq_topk_select(ctx, scores: torch.Tensor, cu_prompt, k_keep, idx_out: torch.Tensor, stream=None) -> None:
    cp, cp_p = _i32(cu_prompt)
    kk, kk_p = _i32(k_keep)
    _check(ctx, load_library().dapq_topk_select(ctx, scores.data_ptr(), cp_p, kk_p, len(kk), idx_out.data_ptr(),
                                                _stream(stream)))


def dapq_compact_kv(ctx, k: torch.Tensor, v: torch.Tensor, cu_rows, prompt_len, idx: torch.Tensor, k_keep,
                    k_out: torch.Tensor, v_out: torch.Tensor, stream=None) -> None:
    view = _view(k, v, cu_rows, prompt_len)
    kk, kk_p = _i32(k_keep)
    _check(ctx, load_library().dapq_compact_kv(ctx, C.byref(view), idx.data_ptr(), kk_p, k_out.data_ptr(),
                                               v_out.data_ptr(), _stream(stream)))


def dapq_recall(ctx, idx_gold: torch.Tensor, idx_pred: torch.Tensor, prompt_len, k_keep, recall_out: torch.Tensor,
                stream=None) -> None:
    pl, pl_p = _i32(prompt_len)
    kk, kk_p = _i32(k_keep)
    _check(ctx, load_library().dapq_recall(ctx, idx_gold.data_ptr(), idx_pred.data_ptr(), pl_p, kk_p, len(kk),
                                           recall_out.data_ptr(), _stream(stream)))


def dapq_evict(ctx, q_pre: torch.Tensor, k: torch.Tensor, v: torch.Tensor, cu_rows, prompt_len, k_keep,
               k_out: torch.Tensor, v_out: torch.Tensor, idx_out: Optional[torch.Tensor] = None,
               scores_out: Optional[torch.Tensor] = None, stream=None) -> None:
    view = _view(k, v, cu_rows, prompt_len)
    kk, kk_p = _i32(k_keep)
    _check(ctx, load_library().dapq_evict(ctx, q_pre.data_ptr(), C.byref(view), kk_p, k_out.data_ptr(),
                                          v_out.data_ptr(), _ptr(idx_out), _ptr(scores_out), _stream(stream)))


def dapq_evict_layers(ctx, q_pre: Sequence[torch.Tensor], k: Sequence[torch.Tensor], v: Sequence[torch.Tensor], cu_rows,
                      prompt_len, k_keep, k_out: Sequence[torch.Tensor], v_out: Sequence[torch.Tensor],
                      idx_out: Optional[Sequence[torch.Tensor]] = None, stream=None, host: bool = False) -> None:
    """k_keep: one budget row [batch] for all layers, or one row per layer [n_layers][batch]."""
    n = len(k)
    views = (dapq_cache_view * n)()
    keep_alive = []
    for l in range(n):
        view = _view(k[l], v[l], cu_rows, prompt_len)
        keep_alive.append(view)
        C.memmove(C.byref(views, l * C.sizeof(dapq_cache_view)), C.byref(view), C.sizeof(dapq_cache_view))
    budgets = np.asarray(k_keep, dtype=np.int32)
    assert budgets.ndim == 1 or (budgets.ndim == 2 and budgets.shape[0] == n)
    kk, kk_p = _i32(budgets.reshape(-1))
    stride = budgets.shape[1] if budgets.ndim == 2 else 0
    arr = lambda ts: (C.c_void_p * n)(*[t.data_ptr() for t in ts])
    idx_arr = arr(idx_out) if idx_out is not None else None
    fn = load_library().dapq_evict_layers_host if host else load_library().dapq_evict_layers
    _check(ctx, fn(ctx, n, arr(q_pre), views, kk_p, stride, arr(k_out), arr(v_out), idx_arr, _stream(stream)))


def dapq_evict_layers_host(ctx, q_pre, k, v, cu_rows, prompt_len, k_keep, k_out, v_out, idx_out=None, stream=None) -> None:
    """dapq_evict_layers on host tensors (pinned memory gives full copy speed); returns once the results are there."""
    dapq_evict_layers(ctx, q_pre, k, v, cu_rows, prompt_len, k_keep, k_out, v_out, idx_out, stream, host=True)


def dapq_evict_host(ctx, q_pre: torch.Tensor, k: torch.Tensor, v: torch.Tensor, cu_rows, prompt_len, k_keep,
                    k_out: torch.Tensor, v_out: torch.Tensor, idx_out: Optional[torch.Tensor] = None,
                    stream=None) -> None:
    """All tensors are HOST tensors (pinned for full copy speed); returns after the results landed."""
    for t in (q_pre, k, v, k_out, v_out):
        assert not t.is_cuda
    view = _view(k, v, cu_rows, prompt_len)
    kk, kk_p = _i32(k_keep)
    _check(ctx, load_library().dapq_evict_host(ctx, q_pre.data_ptr(), C.byref(view), kk_p, k_out.data_ptr(),
                                               v_out.data_ptr(), _ptr(idx_out), _stream(stream)))


DAPQ_STATIC_SCRATCH_BYTES = 2 * 1024 * 1024


def dapq_score_static(n_q_heads: int, n_kv_heads: int, n_pseudo: int, dtype: int, q_rot: torch.Tensor,
                      k: torch.Tensor, cu_rows, prompt_len, scores: torch.Tensor, softmax_scale: float = 0.0,
                      head_dim: int = 128, device: int = 0, stream=None) -> None:
    """dapq_score for callers that may not allocate device memory (no context, no workspace:
    the scratch is a fixed array inside the library).  Raises DapqError(DAPQ_ERR_WORKSPACE)
    when the call needs more than DAPQ_STATIC_SCRATCH_BYTES of scratch."""
    sh = dapq_shape(n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, head_dim=head_dim, n_pseudo=n_pseudo,
                    max_batch=len(prompt_len), dtype=dtype, max_total_rows=int(cu_rows[-1]), rope_base=1.0,
                    softmax_scale=softmax_scale)
    view = _view(k, None, cu_rows, prompt_len)
    err = C.create_string_buffer(512)
    st = load_library().dapq_score_static(C.byref(sh), device, q_rot.data_ptr(), C.byref(view), scores.data_ptr(),
                                          _stream(stream), err, len(err))
    if st != DAPQ_OK:
        raise DapqError(st, err.value.decode())
