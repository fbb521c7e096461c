"""ctypes binding of ``libsam_b200.so``: argument marshalling only.

Function names and argument order follow ``include/sam.h``.  Device arguments are torch
tensors (or raw integer addresses); host arguments are numpy arrays.  Every step of the
path runs in the library's kernels - nothing is computed here.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path
from typing import Optional

import numpy as np

_PKG = Path(__file__).resolve().parent
_LIB_PATH = _PKG / "libsam_b200.so"
_lib = None

SAM_K_MAX = 32
SAM_MAX_SEPARATORS = 16
SAM_STATIC_MAX_ROWS = 16384

_vp, _i32, _i64 = C.c_void_p, C.c_int32, C.c_int64

_SIGNATURES = {
    "sam_build": (C.c_int, [_vp, _i64, _vp, _i32, C.POINTER(_vp)]),
    "sam_sizes": (C.c_int, [_vp, C.POINTER(_i64), C.POINTER(_i64), C.POINTER(_i64)]),
    "sam_export": (C.c_int, [_vp] * 7),
    "sam_upload": (C.c_int, [_vp, _vp, _i64, _vp]),
    "sam_free": (None, [_vp]),
    "sam_workspace_bytes": (_i64, [_i32, _i32]),
    "sam_workspace_init": (C.c_int, [_vp, _i64, _vp]),
    "sam_draft": (C.c_int, [_vp, _i32, _vp, _vp, _vp, _i32, _vp, _i32, _i32, _vp, _vp, _vp]),
    "sam_verify": (C.c_int, [_vp, _i64, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _vp]),
    "sam_step": (C.c_int, [_vp, _vp, _i64, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp,
                           _vp, _vp, _i32, _vp, _vp, _vp, _i64, _vp]),
    "sam_verify_ex": (C.c_int, [_vp, _i64, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, C.c_uint32, _vp, _vp, _i64, _vp]),
    "sam_step_ex": (C.c_int, [_vp, _vp, _i64, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp,
                              _vp, _vp, _i32, _vp, _vp, C.c_uint32, _vp, _vp, _i64, _vp]),
    "sam_adaptive_switch": (C.c_int, [_i64, _i64, _i64, _i64]),
    "sam_speculation_pays": (C.c_int, [_vp, _i32, C.c_double]),
    "sam_set_bytes": (_i64, [_i32]),
    "sam_set_create": (C.c_int, [_vp, _i32, _vp, _i64, _vp, C.POINTER(_vp)]),
    "sam_set_refresh": (C.c_int, [_vp, _vp]),
    "sam_set_free": (None, [_vp]),
    "sam_set_renormalize": (C.c_int, [_vp, _i32, _i32, _i32, _vp, _vp, _vp, _vp]),
    "sam_multi_workspace_bytes": (_i64, [_i32, _i32, _i32]),
    "sam_multi_step": (C.c_int, [_vp, _vp, _i64, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp, _vp,
                                 _i32, _vp, _vp, _vp, _vp, _i64, _vp]),
    "sam_multi_draft": (C.c_int, [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _i32, _vp, _i32, _i32, _vp, _vp, _vp, _vp]),
    "sam_argmax_partial": (C.c_int, [_vp, _i64, _i64, _i32, _i32, _vp, _vp]),
    "sam_step_from_keys": (C.c_int, [_vp, _vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp]),
    "sam_verify_static": (C.c_int, [_vp, _i64, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp]),
    "sam_static_status": (C.c_int, [C.POINTER(_i32), _vp]),
    "sam_step_host_staging_bytes": (_i64, [_i64, _i32, _i32, _i32]),
    "sam_step_host": (C.c_int, [_vp, _vp, _i64, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp,
                                _vp, _vp, _i32, _vp, _vp, _vp, _i64, _vp]),
    "sam_step_host_ex": (C.c_int, [_vp, _vp, _i64, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp,
                                   _vp, _vp, _i32, _vp, _vp, C.c_uint32, _vp, _i64, _vp]),
    "sam_workspace_status": (C.c_int, [_vp, _i32, _i32, C.POINTER(_i32), _vp]),
    "sam_set_argmax_variant": (C.c_int, [_i32]),
    "sam_profile_enable": (C.c_int, [_i32]),
    "sam_profile_count": (_i32, []),
    "sam_profile_read": (C.c_int, [_i32, C.POINTER(C.c_float), C.POINTER(C.c_float)]),
    "sam_strerror": (C.c_char_p, [C.c_int]),
    "sam_last_cuda_error": (C.c_int, []),
    "sam_launch_count": (_i64, []),
    "sam_build_growing": (C.c_int, [_vp, _i64, _vp, _i32, _i64, _i32, C.POINTER(_vp)]),
    "sam_extend": (C.c_int, [_vp, _vp, _i64]),
    "sam_extend_async": (C.c_int, [_vp, _vp, _i64]),
    "sam_pending": (C.c_int, [_vp, C.POINTER(_i64), C.POINTER(_i64), C.POINTER(_i64)]),
    "sam_sync": (C.c_int, [_vp, _vp, C.POINTER(_i64)]),
    "sam_renormalize": (C.c_int, [_vp, _i32, _vp, _vp, _vp]),
    "sam_sync_renormalize": (C.c_int, [_vp, _i32, _vp, _vp, _vp, C.POINTER(_i64)]),
    "sam_growing_set_relayout_every": (C.c_int, [_vp, _i64]),
    "sam_update_stats": (C.c_int, [_vp, C.POINTER(_i64), C.POINTER(_i64), C.POINTER(_i64)]),
}


class SamError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = sam_strerror(status)
        if status == -4:
            msg += f" (cudaError {sam_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{status}]")


def library_path() -> Path:
    return _LIB_PATH


def use_library(path) -> None:
    """Points the binding at another build of this same library (a tuning run comparing two builds, a test
    of the missing-library error).  Only before the first call has loaded the default one."""
    global _LIB_PATH
    if _lib is not None:
        raise RuntimeError("the library is already loaded")
    _LIB_PATH = Path(path)


def exported_symbols():
    """Names every build of the library must export (those declared in include/sam.h)."""
    return list(_SIGNATURES)


def _load():
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise RuntimeError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2512_18337_b200.build` "
                "(there is no CPU fallback)")
        lib = C.CDLL(str(_LIB_PATH))
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def _dev(t) -> Optional[int]:
    """Device address of a torch tensor (must be contiguous, on CUDA) or a raw int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    return t.data_ptr()


def _host(a: Optional[np.ndarray], dtype) -> Optional[int]:
    if a is None:
        return None
    if a.dtype != dtype or not a.flags.c_contiguous:
        raise ValueError(f"expected a contiguous {np.dtype(dtype).name} array")
    return a.ctypes.data


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def _check(status: int, where: str) -> None:
    if status != 0:
        raise SamError(status, where)


# ------------------------------------------------------------------ setup
def sam_build(corpus: np.ndarray, separators) -> int:
    """Host build; returns the opaque handle (release with sam_free)."""
    corpus = np.ascontiguousarray(corpus, dtype=np.int32)
    seps = np.ascontiguousarray(np.atleast_1d(separators), dtype=np.int32)
    h = _vp()
    _check(_load().sam_build(corpus.ctypes.data, corpus.shape[0], seps.ctypes.data if seps.size else None,
                             seps.shape[0], C.byref(h)), "sam_build")
    return h.value


def sam_build_growing(corpus: np.ndarray, separators, max_tokens: int, max_token_id: int) -> int:
    """Host build of an index that can grow (sam_extend); returns the opaque handle."""
    corpus = np.ascontiguousarray(corpus, dtype=np.int32)
    seps = np.ascontiguousarray(np.atleast_1d(separators), dtype=np.int32)
    h = _vp()
    _check(_load().sam_build_growing(corpus.ctypes.data if corpus.size else None, corpus.shape[0],
                                     seps.ctypes.data if seps.size else None, seps.shape[0],
                                     max_tokens, max_token_id, C.byref(h)), "sam_build_growing")
    return h.value


def sam_extend(handle: int, tokens: np.ndarray, wait: bool = True) -> None:
    """Appends host tokens; wait=False only queues them for the builder thread (sam_extend_async)."""
    t = np.ascontiguousarray(tokens, dtype=np.int32)
    fn = _load().sam_extend if wait else _load().sam_extend_async
    _check(fn(handle, t.ctypes.data if t.size else None, t.shape[0]), "sam_extend" if wait else "sam_extend_async")


def sam_pending(handle: int):
    """(tokens_queued, tokens_built, tokens_on_device)."""
    a, b, c = _i64(), _i64(), _i64()
    _check(_load().sam_pending(handle, C.byref(a), C.byref(b), C.byref(c)), "sam_pending")
    return a.value, b.value, c.value


def sam_sync(handle: int, stream=None) -> int:
    """Applies finished updates to the device copy; returns the tokens visible on the device."""
    n = _i64()
    _check(_load().sam_sync(handle, _stream(stream), C.byref(n)), "sam_sync")
    return int(n.value)


def sam_sync_renormalize(handle: int, B: int, state, matched_len, stream=None) -> int:
    """sam_sync and sam_renormalize in one call (one kernel when the pending update is small); returns the
    tokens visible on the device."""
    n = _i64()
    _check(_load().sam_sync_renormalize(handle, B, _dev(state), _dev(matched_len), _stream(stream), C.byref(n)),
           "sam_sync_renormalize")
    return int(n.value)


def sam_update_stats(handle: int):
    """(incremental updates, whole-image updates, bytes copied) applied by sam_sync so far."""
    a, b, c = _i64(), _i64(), _i64()
    _check(_load().sam_update_stats(handle, C.byref(a), C.byref(b), C.byref(c)), "sam_update_stats")
    return a.value, b.value, c.value


def sam_growing_set_relayout_every(handle: int, every: int) -> None:
    """Every `every`-th update of a growing index is sent as a whole image (0: only when it has to be)."""
    _check(_load().sam_growing_set_relayout_every(handle, every), "sam_growing_set_relayout_every")


def sam_renormalize(handle: int, B: int, state, matched_len, stream=None) -> None:
    _check(_load().sam_renormalize(handle, B, _dev(state), _dev(matched_len), _stream(stream)), "sam_renormalize")


def sam_sizes(handle: int):
    """(n_states, n_edges, device_bytes)."""
    a, b, c = _i64(), _i64(), _i64()
    _check(_load().sam_sizes(handle, C.byref(a), C.byref(b), C.byref(c)), "sam_sizes")
    return a.value, b.value, c.value


def sam_export(handle: int):
    """Flat host arrays of the automaton as a dict of numpy arrays."""
    S, E, _ = sam_sizes(handle)
    out = dict(len=np.empty(S, np.int32), link=np.empty(S, np.int32), firstpos=np.empty(S, np.int32),
               row_ptr=np.empty(S + 1, np.int64), edge_tok=np.empty(E, np.int32), edge_dst=np.empty(E, np.int32))
    _check(_load().sam_export(handle, out["len"].ctypes.data, out["link"].ctypes.data,
                              out["firstpos"].ctypes.data, out["row_ptr"].ctypes.data,
                              out["edge_tok"].ctypes.data, out["edge_dst"].ctypes.data), "sam_export")
    return out


def sam_upload(handle: int, device_buf, nbytes: Optional[int] = None, stream=None) -> None:
    nbytes = device_buf.numel() * device_buf.element_size() if nbytes is None else nbytes
    _check(_load().sam_upload(handle, _dev(device_buf), nbytes, _stream(stream)), "sam_upload")


def sam_free(handle: int) -> None:
    _load().sam_free(handle)


def sam_workspace_bytes(B: int, K: int) -> int:
    n = _load().sam_workspace_bytes(B, K)
    if n < 0:
        raise SamError(int(n), "sam_workspace_bytes")
    return int(n)


def sam_workspace_init(workspace, nbytes: Optional[int] = None, stream=None) -> None:
    nbytes = workspace.numel() * workspace.element_size() if nbytes is None else nbytes
    _check(_load().sam_workspace_init(_dev(workspace), nbytes, _stream(stream)), "sam_workspace_init")


# ------------------------------------------------------------------ hot path
def sam_draft(handle, B, state, matched_len, new_tokens, ld, n_new, K, min_match, drafts, n_draft, stream=None):
    _check(_load().sam_draft(handle, B, _dev(state), _dev(matched_len), _dev(new_tokens), ld, _dev(n_new),
                             K, min_match, _dev(drafts), _dev(n_draft), _stream(stream)), "sam_draft")


def sam_verify(logits, row_stride, B, K, V, drafts, n_draft, argmax_out, accepted, n_accepted,
               workspace, workspace_bytes, stream=None):
    _check(_load().sam_verify(_dev(logits), row_stride, B, K, V, _dev(drafts), _dev(n_draft), _dev(argmax_out),
                              _dev(accepted), _dev(n_accepted), _dev(workspace), workspace_bytes,
                              _stream(stream)), "sam_verify")


def sam_verify_static(logits, row_stride, B, K, V, drafts, n_draft, argmax_out, accepted, n_accepted, stream=None):
    """sam_verify for callers that cannot allocate device scratch (an engine plugin whose host has
    already claimed all device memory, or code that only holds foreign raw pointers): the scratch is
    a fixed array inside the library, so B*(K+1) <= SAM_STATIC_MAX_ROWS and calls on one GPU must
    not overlap.  Same outputs as sam_verify."""
    _check(_load().sam_verify_static(_dev(logits), row_stride, B, K, V, _dev(drafts), _dev(n_draft),
                                     _dev(argmax_out), _dev(accepted), _dev(n_accepted), _stream(stream)),
           "sam_verify_static")


def sam_static_status(stream=None) -> int:
    """Status word of the last sam_verify_static call on the current device (0 = completed normally)."""
    out = _i32(0)
    _check(_load().sam_static_status(C.byref(out), _stream(stream)), "sam_static_status")
    return int(out.value)


def sam_step(handle, logits, row_stride, B, K, V, drafts, n_draft, argmax_out, accepted, n_accepted,
             state, matched_len, min_match, next_drafts, next_n_draft, workspace, workspace_bytes, stream=None):
    _check(_load().sam_step(handle, _dev(logits), row_stride, B, K, V, _dev(drafts), _dev(n_draft),
                            _dev(argmax_out), _dev(accepted), _dev(n_accepted), _dev(state), _dev(matched_len),
                            min_match, _dev(next_drafts), _dev(next_n_draft), _dev(workspace), workspace_bytes,
                            _stream(stream)), "sam_step")


SAM_STEP_NO_SPECULATION = 1
SAM_STEP_SKIP_UNUSED_ROWS = 2
SAM_STEP_ROW_LIST_READY = 4
SAM_N_COUNTERS = 6


def sam_verify_ex(logits, row_stride, B, K, V, drafts, n_draft, argmax_out, accepted, n_accepted,
                  flags, counters, workspace, workspace_bytes, stream=None):
    """sam_verify with step options (SAM_STEP_*) and optional device counters (int64[SAM_N_COUNTERS])."""
    _check(_load().sam_verify_ex(_dev(logits), row_stride, B, K, V, _dev(drafts), _dev(n_draft), _dev(argmax_out),
                                 _dev(accepted), _dev(n_accepted), flags, _dev(counters), _dev(workspace),
                                 workspace_bytes, _stream(stream)), "sam_verify_ex")


def sam_step_ex(handle, logits, row_stride, B, K, V, drafts, n_draft, argmax_out, accepted, n_accepted,
                state, matched_len, min_match, next_drafts, next_n_draft, flags, counters,
                workspace, workspace_bytes, stream=None):
    """sam_step with step options (SAM_STEP_*) and optional device counters (int64[SAM_N_COUNTERS])."""
    _check(_load().sam_step_ex(handle, _dev(logits), row_stride, B, K, V, _dev(drafts), _dev(n_draft),
                               _dev(argmax_out), _dev(accepted), _dev(n_accepted), _dev(state), _dev(matched_len),
                               min_match, _dev(next_drafts), _dev(next_n_draft), flags, _dev(counters),
                               _dev(workspace), workspace_bytes, _stream(stream)), "sam_step_ex")


def sam_argmax_partial(logits, row_stride, rows, V, v_offset, keys, stream=None):
    """Packed per-row argmax words of a vocabulary shard (columns v_offset.. of the full vocabulary);
    keys: int64[rows + 1] device tensor (last word = status)."""
    _check(_load().sam_argmax_partial(_dev(logits), row_stride, rows, V, v_offset, _dev(keys), _stream(stream)),
           "sam_argmax_partial")


def sam_step_from_keys(handle, keys, B, K, drafts, n_draft, argmax_out, accepted, n_accepted,
                       state, matched_len, min_match, next_drafts, next_n_draft, stream=None):
    _check(_load().sam_step_from_keys(handle, _dev(keys), B, K, _dev(drafts), _dev(n_draft), _dev(argmax_out),
                                      _dev(accepted), _dev(n_accepted), _dev(state), _dev(matched_len), min_match,
                                      _dev(next_drafts), _dev(next_n_draft), _stream(stream)), "sam_step_from_keys")


class SamSet:
    """A table of uploaded indexes for composite drafting (owns the small device table)."""

    def __init__(self, indexes, device="cuda:0", stream=None):
        import torch
        self.indexes = list(indexes)                      # keeps the members alive
        n = len(self.indexes)
        nbytes = _load().sam_set_bytes(n)
        self.table = torch.empty(nbytes, dtype=torch.uint8, device=device)
        arr = (_vp * n)(*[ix.handle for ix in self.indexes])
        h = _vp()
        _check(_load().sam_set_create(arr, n, _dev(self.table), nbytes, _stream(stream), C.byref(h)), "sam_set_create")
        self.handle = h.value

    def refresh(self, stream=None):
        _check(_load().sam_set_refresh(self.handle, _stream(stream)), "sam_set_refresh")

    def renormalize(self, member: int, B: int, M: int, slots, state, matched_len, stream=None):
        """After member `member` has grown and refresh() was called: repair the slots that name it."""
        _check(_load().sam_set_renormalize(self.handle, member, B, M, _dev(slots), _dev(state), _dev(matched_len),
                                           _stream(stream)), "sam_set_renormalize")

    def close(self):
        h, self.handle = self.handle, None
        if h:
            _load().sam_set_free(h)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def sam_multi_draft(set_handle, B, M, slots, weights, state, matched_len, new_tokens, ld, n_new, K, min_match,
                    drafts, n_draft, chosen, stream=None):
    _check(_load().sam_multi_draft(set_handle, B, M, _dev(slots), _dev(weights), _dev(state), _dev(matched_len),
                                   _dev(new_tokens), ld, _dev(n_new), K, min_match, _dev(drafts), _dev(n_draft),
                                   _dev(chosen), _stream(stream)), "sam_multi_draft")


def sam_multi_workspace_bytes(B: int, K: int, M: int) -> int:
    n = _load().sam_multi_workspace_bytes(B, K, M)
    if n < 0:
        raise SamError(int(n), "sam_multi_workspace_bytes")
    return int(n)


def sam_multi_step(set_handle, logits, row_stride, B, K, V, drafts, n_draft, argmax_out, accepted, n_accepted,
                   M, slots, weights, state, matched_len, min_match, next_drafts, next_n_draft, chosen,
                   workspace, workspace_bytes, stream=None):
    _check(_load().sam_multi_step(set_handle, _dev(logits), row_stride, B, K, V, _dev(drafts), _dev(n_draft),
                                  _dev(argmax_out), _dev(accepted), _dev(n_accepted), M, _dev(slots), _dev(weights),
                                  _dev(state), _dev(matched_len), min_match, _dev(next_drafts), _dev(next_n_draft),
                                  _dev(chosen), _dev(workspace), workspace_bytes, _stream(stream)), "sam_multi_step")


def sam_adaptive_switch(context_len: int, batch_size: int, max_context_len: int, max_batch_size: int) -> bool:
    return bool(_load().sam_adaptive_switch(context_len, batch_size, max_context_len, max_batch_size))


def sam_speculation_pays(counters, K: int, cost_ratio: float) -> bool:
    """Counter-driven switch; `counters` is a HOST int64[SAM_N_COUNTERS] array (a copy of the device counters)."""
    c = np.ascontiguousarray(counters, dtype=np.int64)
    if c.shape != (SAM_N_COUNTERS,):
        raise ValueError("expected SAM_N_COUNTERS int64 values")
    r = _load().sam_speculation_pays(c.ctypes.data, K, float(cost_ratio))
    if r < 0:
        raise SamError(int(r), "sam_speculation_pays")
    return bool(r)


def _hostptr(a) -> Optional[int]:
    """Host address of a numpy array or a CPU torch tensor (contiguous)."""
    if a is None:
        return None
    if isinstance(a, np.ndarray):
        if not a.flags.c_contiguous:
            raise ValueError("expected a contiguous array")
        return a.ctypes.data
    if a.is_cuda or not a.is_contiguous():
        raise ValueError("expected a contiguous host tensor")
    return a.data_ptr()


def sam_step_host_staging_bytes(row_stride: int, B: int, K: int, V: int) -> int:
    n = _load().sam_step_host_staging_bytes(row_stride, B, K, V)
    if n < 0:
        raise SamError(int(n), "sam_step_host_staging_bytes")
    return int(n)


def sam_step_host(handle, logits, row_stride, B, K, V, drafts, n_draft, argmax_out, accepted, n_accepted,
                  state, matched_len, min_match, next_drafts, next_n_draft, staging, staging_bytes, stream=None):
    """All arrays are HOST memory (numpy or CPU torch tensors) except `staging` (device)."""
    _check(_load().sam_step_host(handle, _hostptr(logits), row_stride, B, K, V, _hostptr(drafts), _hostptr(n_draft),
                                 _hostptr(argmax_out), _hostptr(accepted), _hostptr(n_accepted), _hostptr(state),
                                 _hostptr(matched_len), min_match, _hostptr(next_drafts), _hostptr(next_n_draft),
                                 _dev(staging), staging_bytes, _stream(stream)), "sam_step_host")


def sam_step_host_ex(handle, logits, row_stride, B, K, V, drafts, n_draft, argmax_out, accepted, n_accepted,
                     state, matched_len, min_match, next_drafts, next_n_draft, flags, staging, staging_bytes, stream=None):
    """sam_step_host with step options; with SAM_STEP_SKIP_UNUSED_ROWS only the used rows are copied."""
    _check(_load().sam_step_host_ex(handle, _hostptr(logits), row_stride, B, K, V, _hostptr(drafts), _hostptr(n_draft),
                                    _hostptr(argmax_out), _hostptr(accepted), _hostptr(n_accepted), _hostptr(state),
                                    _hostptr(matched_len), min_match, _hostptr(next_drafts), _hostptr(next_n_draft),
                                    flags, _dev(staging), staging_bytes, _stream(stream)), "sam_step_host_ex")


def sam_workspace_status(workspace, B: int, K: int, stream=None) -> int:
    out = _i32(0)
    _check(_load().sam_workspace_status(_dev(workspace), B, K, C.byref(out), _stream(stream)), "sam_workspace_status")
    return int(out.value)


def sam_set_argmax_variant(variant: int) -> None:
    _check(_load().sam_set_argmax_variant(variant), "sam_set_argmax_variant")


def sam_profile_enable(max_calls: int) -> None:
    _check(_load().sam_profile_enable(max_calls), "sam_profile_enable")


def sam_profile_count() -> int:
    return int(_load().sam_profile_count())


def sam_profile_read(call: int):
    """(argmax_ms, accept_ms) of the call-th profiled sam_verify / sam_step."""
    a, b = C.c_float(), C.c_float()
    _check(_load().sam_profile_read(call, C.byref(a), C.byref(b)), "sam_profile_read")
    return a.value, b.value


def sam_strerror(status: int) -> str:
    return _load().sam_strerror(status).decode()


def sam_last_cuda_error() -> int:
    return int(_load().sam_last_cuda_error())


def sam_launch_count() -> int:
    return int(_load().sam_launch_count())


# ------------------------------------------------------------------ convenience holder
class SamIndex:
    """Owns a built handle and the torch tensor that holds its device blob (memory plumbing only)."""

    def __init__(self, corpus: np.ndarray, separators, device="cuda:0", upload: bool = True,
                 max_tokens: Optional[int] = None, max_token_id: Optional[int] = None):
        """max_tokens given: an index that can grow up to that many tokens (sam_build_growing)."""
        if max_tokens is None:
            self.handle = sam_build(corpus, separators)
        else:
            self.handle = sam_build_growing(corpus, separators, max_tokens, max_token_id)
        self.n_states, self.n_edges, self.device_bytes = sam_sizes(self.handle)
        self.blob = None
        if upload:
            import torch
            self.blob = torch.empty(self.device_bytes, dtype=torch.uint8, device=device)
            sam_upload(self.handle, self.blob)

    def close(self):
        h, self.handle = self.handle, None
        if h:
            sam_free(h)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
