"""Thin ctypes binding of liblookm.so: same names as the C ABI, argument marshalling only.

Device buffers are torch CUDA tensors (PyTorch is used for device memory and streams, nothing
else); host arrays are Python sequences of ints.  Every function returns the library's status
code unless stated otherwise and raises nothing for device-side results; :func:`check` turns a
non-zero status into an exception.  Loading fails loudly if the library has not been built:
there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblookm.so")     # the in-tree build, nothing else
_lib = None

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE_TOO_SMALL, ERR_CUDA, ERR_DEVICE_TIMEOUT, \
    ERR_DEVICE_BAD_INDEX = range(7)
MERGE_AVERAGE, MERGE_PIVOTAL, MERGE_WEIGHTED, MERGE_NONE = 0, 1, 2, 3
OPT_NO_TEXT_PRIOR = 1

EXPORTS = ["lookm_workspace_size", "lookm_workspace_layout", "lookm_compress_layer", "lookm_compress_varlen",
           "lookm_compress_layer_opt", "lookm_compress_varlen_opt", "lookm_score",
           "lookm_select", "lookm_match", "lookm_match_from_sim", "lookm_merge",
           "lookm_decode_workspace_size", "lookm_decode_step", "lookm_decode_step_varlen",
           "lookm_set_stage_events", "lookm_selftest_wait_expiry", "lookm_merge_noalloc", "lookm_noalloc_status", "lookm_device_status", "lookm_last_launch_count", "lookm_strerror"]
N_STAGE_EVENTS = 8
STAGE_NAMES = ["score_sweep1", "score_sweep2", "select_norms", "gather", "match", "invert", "merge"]


class WorkspaceOffsets(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in ("status", "lse", "scores", "rank", "kept_idx", "evict_idx",
                                          "assign", "sim")]


class Options(C.Structure):
    _fields_ = [("flags", C.c_uint), ("lse", C.c_void_p), ("out_stride_head", C.c_longlong)]


class CacheLayout(C.Structure):
    _fields_ = [("n_q_heads", C.c_int), ("n_kv_heads", C.c_int), ("head_dim", C.c_int),
                ("cache_stride_row", C.c_longlong), ("cache_stride_head", C.c_longlong),
                ("softmax_scale", C.c_float)]


class Layout(C.Structure):
    _fields_ = [("n_q_heads", C.c_int), ("n_kv_heads", C.c_int), ("head_dim", C.c_int),
                ("q_stride_tok", C.c_longlong), ("q_stride_head", C.c_longlong),
                ("kv_stride_tok", C.c_longlong), ("kv_stride_head", C.c_longlong),
                ("softmax_scale", C.c_float)]


def lib():
    """The loaded library; raises if liblookm.so is missing (build it with build.py)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("liblookm.so is not built: run `python -m paper_2406_18139_b200.build` "
                               "(there is no CPU or eager fallback)")
        L = C.CDLL(LIB_PATH)
        vp, ip, sz = C.c_void_p, C.POINTER(C.c_int), C.c_size_t
        lp = C.POINTER(Layout)
        L.lookm_workspace_size.argtypes = [lp, C.c_int, ip, ip]
        L.lookm_workspace_size.restype = sz
        L.lookm_workspace_layout.argtypes = [lp, C.c_int, ip, C.POINTER(WorkspaceOffsets)]
        L.lookm_workspace_layout.restype = C.c_int
        L.lookm_compress_layer.argtypes = [vp, vp, vp, vp, C.c_int, C.c_int, C.c_int, C.c_int, lp,
                                           vp, vp, ip, vp, sz, vp]
        L.lookm_compress_varlen.argtypes = [vp, vp, vp, vp, ip, C.c_int, ip, ip, ip, lp, vp, vp, ip,
                                            vp, sz, vp]
        op = C.POINTER(Options)
        L.lookm_compress_layer_opt.argtypes = [vp, vp, vp, vp, C.c_int, C.c_int, C.c_int, C.c_int, lp, op,
                                               vp, vp, ip, vp, sz, vp]
        L.lookm_compress_varlen_opt.argtypes = [vp, vp, vp, vp, ip, C.c_int, ip, ip, ip, lp, op, vp, vp, ip,
                                                vp, sz, vp]
        cp = C.POINTER(CacheLayout)
        L.lookm_decode_workspace_size.argtypes = [cp, C.c_int, ip]
        L.lookm_decode_workspace_size.restype = sz
        L.lookm_decode_step.argtypes = [vp, vp, vp, vp, vp, C.c_int, cp, vp, vp, sz, vp]
        L.lookm_decode_step.restype = C.c_int
        L.lookm_decode_step_varlen.argtypes = [vp, vp, vp, vp, vp, C.POINTER(C.c_longlong), ip, C.c_int, cp,
                                               vp, vp, sz, vp]
        L.lookm_decode_step_varlen.restype = C.c_int
        L.lookm_score.argtypes = [vp, vp, ip, C.c_int, lp, vp, vp, C.c_int, vp, sz, vp]
        L.lookm_select.argtypes = [vp, vp, ip, C.c_int, ip, ip, C.c_int, vp, vp, vp, vp, sz, vp]
        L.lookm_match.argtypes = [vp, vp, vp, ip, C.c_int, ip, lp, vp, vp, vp, sz, vp]
        L.lookm_match_from_sim.argtypes = [vp, ip, C.c_int, ip, C.c_int, vp, vp, vp, sz, vp]
        L.lookm_merge.argtypes = [vp, vp, vp, vp, vp, vp, ip, C.c_int, ip, ip, lp, C.c_int, vp, vp,
                                  vp, sz, vp]
        L.lookm_set_stage_events.argtypes = [C.POINTER(C.c_void_p), C.c_int]
        L.lookm_set_stage_events.restype = C.c_int
        L.lookm_selftest_wait_expiry.argtypes = [C.c_int, vp, sz, vp]
        L.lookm_selftest_wait_expiry.restype = C.c_int
        L.lookm_merge_noalloc.argtypes = [vp, vp, vp, vp, vp, vp, ip, C.c_int, ip, ip, lp, C.c_int, vp, vp, vp]
        L.lookm_merge_noalloc.restype = C.c_int
        L.lookm_noalloc_status.argtypes = [vp]
        L.lookm_noalloc_status.restype = C.c_int
        L.lookm_device_status.argtypes = [vp, vp]
        L.lookm_last_launch_count.argtypes = []
        L.lookm_strerror.argtypes = [C.c_int]
        L.lookm_strerror.restype = C.c_char_p
        for name in ("lookm_compress_layer", "lookm_compress_varlen", "lookm_compress_layer_opt",
                     "lookm_compress_varlen_opt", "lookm_score", "lookm_select",
                     "lookm_match", "lookm_match_from_sim", "lookm_merge", "lookm_device_status",
                     "lookm_last_launch_count"):
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def _ints(seq: Optional[Sequence[int]]):
    if seq is None:
        return None
    seq = [int(x) for x in seq]
    return (C.c_int * len(seq))(*seq)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def lookm_strerror(status: int) -> str:
    return lib().lookm_strerror(int(status)).decode()


def check(status: int) -> None:
    if status != OK:
        raise RuntimeError("lookm: %s (status %d)" % (lookm_strerror(status), status))


def make_layout(q, k, softmax_scale: float = 0.0) -> Layout:
    """Layout of Q [T, Hq, 128] and K/V [T, Hkv, 128] tensors (any strides, last dim contiguous)."""
    assert k.stride(2) == 1 and (q is None or q.stride(2) == 1)
    qq = q if q is not None else k
    return Layout(qq.shape[1], k.shape[1], k.shape[2], qq.stride(0), qq.stride(1), k.stride(0),
                  k.stride(1), float(softmax_scale))


def lookm_workspace_size(layout: Layout, seq_lens: Sequence[int], budgets: Optional[Sequence[int]] = None) -> int:
    return int(lib().lookm_workspace_size(C.byref(layout), len(seq_lens), _ints(seq_lens), _ints(budgets)))


def lookm_workspace_layout(layout: Layout, seq_lens: Sequence[int]) -> WorkspaceOffsets:
    off = WorkspaceOffsets()
    check(lib().lookm_workspace_layout(C.byref(layout), len(seq_lens), _ints(seq_lens), C.byref(off)))
    return off


def read_intermediates(workspace, layout: Layout, seq_lens: Sequence[int], budgets: Sequence[int]):
    """Copies the intermediate results of the last whole-path call out of the workspace.

    Returns (scores [Hkv, T] float32, per_request) where per_request[r][h] is the tuple
    (kept positions, evicted positions, assign, sim) of request r and KV head h as numpy arrays.
    """
    import numpy as np
    import torch
    torch.cuda.synchronize()
    off = lookm_workspace_layout(layout, seq_lens)
    Hkv, T = layout.n_kv_heads, int(sum(seq_lens))
    Bs = [min(int(b), int(L)) for b, L in zip(budgets, seq_lens)]
    Es = [int(L) - b for b, L in zip(Bs, seq_lens)]

    def view(byte_off, count, dtype):
        nbytes = count * 4
        return workspace[byte_off:byte_off + nbytes].view(dtype).cpu().numpy()

    scores = view(off.scores, Hkv * T, torch.float32).reshape(Hkv, T)
    kept = view(off.kept_idx, Hkv * sum(Bs), torch.int32)
    ev = view(off.evict_idx, Hkv * sum(Es), torch.int32)
    asg = view(off.assign, Hkv * sum(Es), torch.int32)
    sim = view(off.sim, Hkv * sum(Es), torch.float32)
    per_request, ko, eo = [], 0, 0
    for b, e in zip(Bs, Es):
        heads = []
        for h in range(Hkv):
            heads.append((kept[ko + h * b: ko + (h + 1) * b], ev[eo + h * e: eo + (h + 1) * e],
                          asg[eo + h * e: eo + (h + 1) * e], sim[eo + h * e: eo + (h + 1) * e]))
        per_request.append(heads)
        ko += Hkv * b
        eo += Hkv * e
    return scores, per_request


def make_options(no_text_prior: bool = False, lse=None, out_stride_head: int = 0) -> Options:
    """Options of the *_opt calls; `lse` is a float32 CUDA tensor [n_q_heads, total_tokens] or None
    (the caller keeps it alive until the call's work has run)."""
    return Options(OPT_NO_TEXT_PRIOR if no_text_prior else 0, None if lse is None else lse.data_ptr(),
                   int(out_stride_head))


def lookm_compress_layer(q, k, v, modality_mask, seq_len, budget, recent_window, merge_mode, layout,
                         out_k, out_v, workspace, stream=None):
    """Returns (status, out_len)."""
    out_len = C.c_int(0)
    st = lib().lookm_compress_layer(_ptr(q), _ptr(k), _ptr(v), _ptr(modality_mask), int(seq_len),
                                    int(budget), int(recent_window), int(merge_mode), C.byref(layout),
                                    _ptr(out_k), _ptr(out_v), C.byref(out_len), _ptr(workspace),
                                    workspace.numel() * workspace.element_size(), _stream(stream))
    return st, out_len.value


def lookm_compress_layer_opt(q, k, v, modality_mask, seq_len, budget, recent_window, merge_mode, layout,
                             options, out_k, out_v, workspace, stream=None):
    """Returns (status, out_len).  options: an Options (see make_options) or None."""
    out_len = C.c_int(0)
    st = lib().lookm_compress_layer_opt(_ptr(q), _ptr(k), _ptr(v), _ptr(modality_mask), int(seq_len),
                                        int(budget), int(recent_window), int(merge_mode), C.byref(layout),
                                        None if options is None else C.byref(options), _ptr(out_k),
                                        _ptr(out_v), C.byref(out_len), _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), _stream(stream))
    return st, out_len.value


def lookm_compress_varlen(q, k, v, modality_mask, cu_seqlens, budgets, windows, merge_modes, layout,
                          out_k, out_v, workspace, stream=None):
    """Returns (status, out_cu_seqlens list)."""
    n = len(cu_seqlens) - 1
    out_cu = (C.c_int * (n + 1))()
    st = lib().lookm_compress_varlen(_ptr(q), _ptr(k), _ptr(v), _ptr(modality_mask), _ints(cu_seqlens),
                                     n, _ints(budgets), _ints(windows), _ints(merge_modes),
                                     C.byref(layout), _ptr(out_k), _ptr(out_v), out_cu, _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _stream(stream))
    return st, list(out_cu)


def lookm_compress_varlen_opt(q, k, v, modality_mask, cu_seqlens, budgets, windows, merge_modes, layout,
                              options, out_k, out_v, workspace, stream=None):
    """Returns (status, out_cu_seqlens list).  options: an Options (see make_options) or None."""
    n = len(cu_seqlens) - 1
    out_cu = (C.c_int * (n + 1))()
    st = lib().lookm_compress_varlen_opt(_ptr(q), _ptr(k), _ptr(v), _ptr(modality_mask), _ints(cu_seqlens),
                                         n, _ints(budgets), _ints(windows), _ints(merge_modes),
                                         C.byref(layout), None if options is None else C.byref(options),
                                         _ptr(out_k), _ptr(out_v), out_cu, _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _stream(stream))
    return st, list(out_cu)


def lookm_score(q, k, cu_seqlens, layout, scores, lse, lse_is_input, workspace, stream=None):
    return lib().lookm_score(_ptr(q), _ptr(k), _ints(cu_seqlens), len(cu_seqlens) - 1, C.byref(layout),
                             _ptr(scores), _ptr(lse), int(bool(lse_is_input)), _ptr(workspace),
                             workspace.numel() * workspace.element_size(), _stream(stream))


def lookm_select(scores, modality_mask, cu_seqlens, budgets, windows, n_kv_heads, kept_idx, evict_idx,
                 rank, workspace, stream=None):
    return lib().lookm_select(_ptr(scores), _ptr(modality_mask), _ints(cu_seqlens), len(cu_seqlens) - 1,
                              _ints(budgets), _ints(windows), int(n_kv_heads), _ptr(kept_idx),
                              _ptr(evict_idx), _ptr(rank), _ptr(workspace),
                              workspace.numel() * workspace.element_size(), _stream(stream))


def lookm_match(k, kept_idx, evict_idx, cu_seqlens, budgets, layout, assign, sim, workspace, stream=None):
    return lib().lookm_match(_ptr(k), _ptr(kept_idx), _ptr(evict_idx), _ints(cu_seqlens),
                             len(cu_seqlens) - 1, _ints(budgets), C.byref(layout), _ptr(assign),
                             _ptr(sim), _ptr(workspace), workspace.numel() * workspace.element_size(),
                             _stream(stream))


def lookm_match_from_sim(sim_matrix, cu_seqlens, budgets, n_kv_heads, assign, sim, workspace, stream=None):
    return lib().lookm_match_from_sim(_ptr(sim_matrix), _ints(cu_seqlens), len(cu_seqlens) - 1,
                                      _ints(budgets), int(n_kv_heads), _ptr(assign), _ptr(sim),
                                      _ptr(workspace), workspace.numel() * workspace.element_size(),
                                      _stream(stream))


def lookm_merge(k, v, kept_idx, evict_idx, assign, sim, cu_seqlens, budgets, merge_modes, layout,
                varlen_output, out_k, out_v, workspace, stream=None):
    return lib().lookm_merge(_ptr(k), _ptr(v), _ptr(kept_idx), _ptr(evict_idx), _ptr(assign), _ptr(sim),
                             _ints(cu_seqlens), len(cu_seqlens) - 1, _ints(budgets), _ints(merge_modes),
                             C.byref(layout), int(bool(varlen_output)), _ptr(out_k), _ptr(out_v),
                             _ptr(workspace), workspace.numel() * workspace.element_size(),
                             _stream(stream))


def lookm_merge_noalloc(k, v, kept_idx, evict_idx, assign, sim, cu_seqlens, budgets, merge_modes, layout,
                        varlen_output, out_k, out_v, stream=None):
    """lookm_merge without a workspace argument: the library's built-in scratch array is used, so
    the call allocates nothing (for hosts that may not call cudaMalloc while serving)."""
    return lib().lookm_merge_noalloc(_ptr(k), _ptr(v), _ptr(kept_idx), _ptr(evict_idx), _ptr(assign),
                                     _ptr(sim), _ints(cu_seqlens), len(cu_seqlens) - 1, _ints(budgets),
                                     _ints(merge_modes), C.byref(layout), int(bool(varlen_output)),
                                     _ptr(out_k), _ptr(out_v), _stream(stream))


def lookm_noalloc_status(stream=None) -> int:
    return lib().lookm_noalloc_status(_stream(stream))


def lookm_decode_workspace_size(layout: CacheLayout, cache_lens: Sequence[int]) -> int:
    return int(lib().lookm_decode_workspace_size(C.byref(layout), len(cache_lens), _ints(cache_lens)))


def alloc_decode_workspace(layout: CacheLayout, n_requests: int = 1, device="cuda"):
    import torch
    n = lookm_decode_workspace_size(layout, [0] * n_requests)
    if n == 0:
        raise ValueError("lookm_decode_workspace_size rejected the layout")
    return torch.empty(n, dtype=torch.uint8, device=device)


def lookm_decode_step(q, k_new, v_new, cache_k, cache_v, cache_len, layout: CacheLayout, out, workspace,
                      stream=None):
    return lib().lookm_decode_step(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(cache_k), _ptr(cache_v),
                                   int(cache_len), C.byref(layout), _ptr(out), _ptr(workspace),
                                   workspace.numel() * workspace.element_size(), _stream(stream))


def lookm_decode_step_varlen(q, k_new, v_new, cache_k, cache_v, cache_begin, cache_lens, layout: CacheLayout,
                             out, workspace, stream=None):
    begins = (C.c_longlong * len(cache_begin))(*[int(b) for b in cache_begin])
    return lib().lookm_decode_step_varlen(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(cache_k), _ptr(cache_v),
                                          begins, _ints(cache_lens), len(cache_lens), C.byref(layout),
                                          _ptr(out), _ptr(workspace),
                                          workspace.numel() * workspace.element_size(), _stream(stream))


_stage_event_array = None


def lookm_set_stage_events(events) -> int:
    """events: 8 torch.cuda.Event (created with enable_timing=True and recorded once so that their
    handles exist; an entry may be None to skip that boundary), or None to stop per-stage timing."""
    global _stage_event_array
    if events is None:
        _stage_event_array = None
        return lib().lookm_set_stage_events(None, 0)
    arr = (C.c_void_p * len(events))(*[(e.cuda_event if e is not None else None) for e in events])
    _stage_event_array = arr                     # the library keeps the pointer: keep it alive
    return lib().lookm_set_stage_events(arr, len(events))


def lookm_selftest_wait_expiry(limit_us: int, workspace, stream=None) -> int:
    return lib().lookm_selftest_wait_expiry(int(limit_us), _ptr(workspace),
                                            workspace.numel() * workspace.element_size(), _stream(stream))


def lookm_device_status(workspace, stream=None) -> int:
    return lib().lookm_device_status(_ptr(workspace), _stream(stream))


def lookm_last_launch_count() -> int:
    return lib().lookm_last_launch_count()


def alloc_workspace(layout: Layout, seq_lens: Sequence[int], device="cuda"):
    """A torch uint8 buffer of lookm_workspace_size bytes (torch allocations are 256-byte aligned)."""
    import torch
    n = lookm_workspace_size(layout, seq_lens)
    if n == 0:
        raise ValueError("lookm_workspace_size rejected the layout")
    return torch.empty(n, dtype=torch.uint8, device=device)
