"""Thin ctypes binding of libkvs.so: argument marshalling only.

Every function here has the name of the C entry point it calls (see include/kvs.h) and does
nothing but turn torch tensors / Python lists into pointers and sizes.  There is no
fallback: if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import math
import os
from typing import Dict, List, Optional, Sequence, Tuple

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libkvs.so")
_lib = None

KVS_OK = 0
STATUS_NAMES = {0: "KVS_OK", 1: "KVS_ERR_INVALID_ARG", 2: "KVS_ERR_UNSUPPORTED",
                3: "KVS_ERR_WORKSPACE", 4: "KVS_ERR_BUDGET_UNREACHABLE", 5: "KVS_ERR_CUDA",
                6: "KVS_ERR_TIMEOUT"}

EXPORTS = ["kvs_version", "kvs_last_error_string", "kvs_launch_count", "kvs_round_plan",
           "kvs_workspace_size", "kvs_merge_layer", "kvs_compact", "kvs_decode_attn",
           "kvs_window_stats", "kvs_profile_begin", "kvs_profile_end", "kvs_profile_kind_name",
           "kvs_compact_static", "kvs_static_scratch_bytes", "kvs_append_and_merge",
           "kvs_debug_set_wait", "kvs_adjacent_cosine",
           "kvs_workspace_size_per_head", "kvs_merge_layer_per_head", "kvs_decode_attn_per_head",
           "kvs_merge_layer_exact", "kvs_window_stats_exact", "kvs_probe_sfu", "kvs_probe_mma"]


class KvsError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"{STATUS_NAMES.get(code, code)}: {msg}")
        self.code = code


class kvs_params_t(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
                ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("window", ctypes.c_int32), ("sink", ctypes.c_int32),
                ("recent", ctypes.c_int32), ("causal", ctypes.c_int32),
                ("softmax_scale", ctypes.c_float), ("round_frac", ctypes.c_float),
                ("score_mode", ctypes.c_int32), ("first_round", ctypes.c_int32),
                ("k_stride_b", ctypes.c_int64), ("k_stride_h", ctypes.c_int64),
                ("k_stride_t", ctypes.c_int64), ("v_stride_b", ctypes.c_int64),
                ("v_stride_h", ctypes.c_int64), ("v_stride_t", ctypes.c_int64)]


def lib() -> ctypes.CDLL:
    """Load libkvs.so (built in-tree by build.py).  Raises if it is not there."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2603_00907_b200.build` "
                               "(there is no CPU fallback)")
        L = ctypes.CDLL(_LIB_PATH)
        L.kvs_version.restype = ctypes.c_int
        L.kvs_last_error_string.restype = ctypes.c_char_p
        L.kvs_launch_count.restype = ctypes.c_uint64
        L.kvs_profile_kind_name.restype = ctypes.c_char_p
        L.kvs_profile_kind_name.argtypes = [ctypes.c_int32]
        L.kvs_static_scratch_bytes.restype = ctypes.c_size_t
        for name in ("kvs_round_plan", "kvs_workspace_size", "kvs_merge_layer", "kvs_compact",
                     "kvs_decode_attn", "kvs_window_stats", "kvs_profile_begin", "kvs_profile_end",
                     "kvs_compact_static", "kvs_append_and_merge", "kvs_debug_set_wait", "kvs_adjacent_cosine",
                     "kvs_workspace_size_per_head", "kvs_merge_layer_per_head", "kvs_decode_attn_per_head",
                     "kvs_merge_layer_exact", "kvs_window_stats_exact", "kvs_probe_sfu", "kvs_probe_mma"):
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def _check(code: int) -> None:
    if code != KVS_OK:
        raise KvsError(code, lib().kvs_last_error_string().decode())


def _ptr(t) -> ctypes.c_void_p:
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _i32(values: Sequence[int]):
    return (ctypes.c_int32 * len(values))(*[int(v) for v in values])


def make_params(K, V, n_q_heads: int, window: int, *, sink: int = 32, recent: Optional[int] = None,
                causal: bool = True, softmax_scale: Optional[float] = None,
                round_frac: float = 0.5, score_mode: int = 0, first_round: int = 0) -> kvs_params_t:
    """Parameter block for caches K, V of shape [B, Hkv, Nmax, 128] (element strides are read
    from the tensors)."""
    B, Hkv, _, d = K.shape
    p = kvs_params_t()
    p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim = B, n_q_heads, Hkv, d
    p.window, p.sink = window, sink
    p.recent = window if recent is None else recent
    p.causal = 1 if causal else 0
    p.softmax_scale = 1.0 / math.sqrt(d) if softmax_scale is None else softmax_scale
    p.round_frac, p.score_mode, p.first_round = round_frac, score_mode, first_round
    p.k_stride_b, p.k_stride_h, p.k_stride_t = K.stride(0), K.stride(1), K.stride(2)
    p.v_stride_b, p.v_stride_h, p.v_stride_t = V.stride(0), V.stride(1), V.stride(2)
    return p


def _stream() -> ctypes.c_void_p:
    import torch
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def kvs_version() -> int:
    return lib().kvs_version()


def kvs_launch_count() -> int:
    return int(lib().kvs_launch_count())


def kvs_round_plan(params: kvs_params_t, n: int, budget: int, max_rounds: int = 64
                   ) -> List[Tuple[int, int, int, int]]:
    """[(n_r, off_r, P_r, R_r)] for every round (host only)."""
    n_r, off_r = (ctypes.c_int32 * max_rounds)(), (ctypes.c_int32 * max_rounds)()
    P_r, R_r = (ctypes.c_int32 * max_rounds)(), (ctypes.c_int32 * max_rounds)()
    cnt = ctypes.c_int32(0)
    _check(lib().kvs_round_plan(ctypes.byref(params), n, budget, max_rounds, n_r, off_r, P_r, R_r,
                                ctypes.byref(cnt)))
    return [(n_r[i], off_r[i], P_r[i], R_r[i]) for i in range(cnt.value)]


def kvs_workspace_size(params: kvs_params_t, max_seq_len: int, max_new: int = 0) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().kvs_workspace_size(ctypes.byref(params), max_seq_len, max_new, ctypes.byref(out)))
    return int(out.value)


def kvs_merge_layer(params: kvs_params_t, K, V, counts, q_win, seq_len: Sequence[int],
                    budget: Sequence[int], workspace, status_dev=None) -> List[int]:
    """In-place merge pass of one layer.  Returns new_len per sequence."""
    B = params.batch
    new_len = (ctypes.c_int32 * B)()
    _check(lib().kvs_merge_layer(ctypes.byref(params), _ptr(K), _ptr(V), _ptr(counts), _ptr(q_win),
                                 _i32(seq_len), _i32(budget), ctypes.c_int32(counts.shape[-1]),
                                 new_len, _ptr(workspace),
                                 ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                                 _ptr(status_dev), _stream()))
    return list(new_len)


def kvs_append_and_merge(params: kvs_params_t, K, V, counts, chunk_k, chunk_v, q_win,
                         cur_len: Sequence[int], budget: Sequence[int], workspace,
                         status_dev=None) -> List[int]:
    """One streaming step in place: append the chunk [B,Hkv,chunk_len,128] after the slots in use,
    then merge back to the budget.  Returns new_len per sequence."""
    B = params.batch
    new_len = (ctypes.c_int32 * B)()
    _check(lib().kvs_append_and_merge(ctypes.byref(params), _ptr(K), _ptr(V), _ptr(counts), _ptr(chunk_k),
                                      _ptr(chunk_v), ctypes.c_int32(chunk_k.shape[2]), _ptr(q_win),
                                      _i32(cur_len), _i32(budget), ctypes.c_int32(counts.shape[-1]),
                                      new_len, _ptr(workspace),
                                      ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                                      _ptr(status_dev), _stream()))
    return list(new_len)


def kvs_compact(params: kvs_params_t, K, V, counts, merge_mask, w_left, seq_len: Sequence[int],
                n_merge: Sequence[int], workspace, new_index=None, status_dev=None) -> List[int]:
    B = params.batch
    new_len = (ctypes.c_int32 * B)()
    _check(lib().kvs_compact(ctypes.byref(params), _ptr(K), _ptr(V), _ptr(counts), _ptr(merge_mask),
                             _ptr(w_left), _i32(seq_len), _i32(n_merge),
                             ctypes.c_int32(counts.shape[-1]), new_len, _ptr(new_index),
                             _ptr(workspace),
                             ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                             _ptr(status_dev), _stream()))
    return list(new_len)


def kvs_compact_static(params: kvs_params_t, K, V, counts, merge_mask, w_left, seq_len: Sequence[int],
                       n_merge: Sequence[int], new_index=None, status_dev=None) -> List[int]:
    """kvs_compact for callers that cannot allocate: no workspace argument, the scratch is a fixed
    array inside the library (kvs_static_scratch_bytes()); calls must not overlap on the GPU."""
    B = params.batch
    new_len = (ctypes.c_int32 * B)()
    _check(lib().kvs_compact_static(ctypes.byref(params), _ptr(K), _ptr(V), _ptr(counts),
                                    _ptr(merge_mask), _ptr(w_left), _i32(seq_len), _i32(n_merge),
                                    ctypes.c_int32(counts.shape[-1]), new_len, _ptr(new_index),
                                    _ptr(status_dev), _stream()))
    return list(new_len)


def kvs_static_scratch_bytes() -> int:
    return int(lib().kvs_static_scratch_bytes())


def kvs_decode_attn(params: kvs_params_t, q_new, K, V, counts, seq_len: Sequence[int], out,
                    workspace, lse=None, status_dev=None) -> None:
    n_new = q_new.shape[2]
    _check(lib().kvs_decode_attn(ctypes.byref(params), _ptr(q_new), ctypes.c_int32(n_new), _ptr(K),
                                 _ptr(V), _ptr(counts), _i32(seq_len),
                                 ctypes.c_int32(counts.shape[-1]), _ptr(out), _ptr(lse),
                                 _ptr(workspace),
                                 ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                                 _ptr(status_dev), _stream()))


def kvs_window_stats(params: kvs_params_t, K, V, counts, q_win, seq_len: Sequence[int],
                     budget: Sequence[int], workspace, *, A=None, N1=None, N12=None, cosv=None,
                     score=None, w=None, mask=None, o_win=None, lse_win=None,
                     status_dev=None) -> None:
    _check(lib().kvs_window_stats(ctypes.byref(params), _ptr(K), _ptr(V), _ptr(counts), _ptr(q_win),
                                  _i32(seq_len), _i32(budget), ctypes.c_int32(counts.shape[-1]),
                                  _ptr(A), _ptr(N1), _ptr(N12), _ptr(cosv), _ptr(score), _ptr(w),
                                  _ptr(mask), _ptr(o_win), _ptr(lse_win), _ptr(workspace),
                                  ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                                  _ptr(status_dev), _stream()))


def kvs_merge_layer_exact(params: kvs_params_t, K, V, counts, q_win, e_win, weight_mode: int,
                          seq_len: Sequence[int], budget: Sequence[int], workspace, status_dev=None) -> List[int]:
    """kvs_merge_layer with exact weights from the loss gradient rows e_win [B,Hq,W,128]
    (weight_mode 1) or their diagonal-only form (2)."""
    B = params.batch
    new_len = (ctypes.c_int32 * B)()
    _check(lib().kvs_merge_layer_exact(ctypes.byref(params), _ptr(K), _ptr(V), _ptr(counts), _ptr(q_win),
                                       _ptr(e_win), ctypes.c_int32(weight_mode), _i32(seq_len), _i32(budget),
                                       ctypes.c_int32(counts.shape[-1]), new_len, _ptr(workspace),
                                       ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                                       _ptr(status_dev), _stream()))
    return list(new_len)


def kvs_window_stats_exact(params: kvs_params_t, K, V, counts, q_win, e_win, weight_mode: int,
                           seq_len: Sequence[int], budget: Sequence[int], workspace, *, A=None, g_self=None,
                           g_pair=None, cosv=None, score=None, w=None, mask=None, status_dev=None) -> None:
    _check(lib().kvs_window_stats_exact(ctypes.byref(params), _ptr(K), _ptr(V), _ptr(counts), _ptr(q_win),
                                        _ptr(e_win), ctypes.c_int32(weight_mode), _i32(seq_len), _i32(budget),
                                        ctypes.c_int32(counts.shape[-1]), _ptr(A), _ptr(g_self), _ptr(g_pair),
                                        _ptr(cosv), _ptr(score), _ptr(w), _ptr(mask), _ptr(workspace),
                                        ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                                        _ptr(status_dev), _stream()))


def kvs_workspace_size_per_head(params: kvs_params_t, n_max: int, max_new: int = 0) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().kvs_workspace_size_per_head(ctypes.byref(params), n_max, max_new, ctypes.byref(out)))
    return int(out.value)


def kvs_merge_layer_per_head(params: kvs_params_t, K, V, counts, q_win, seq_len: Sequence[int],
                             budget: Sequence[int], workspace, status_dev=None) -> List[int]:
    """kvs_merge_layer with a length and a budget per (sequence, KV head): flat lists of B * Hkv
    entries, index b * Hkv + h.  Returns new_len in the same order."""
    U = params.batch * params.n_kv_heads
    new_len = (ctypes.c_int32 * U)()
    _check(lib().kvs_merge_layer_per_head(ctypes.byref(params), _ptr(K), _ptr(V), _ptr(counts), _ptr(q_win),
                                          _i32(seq_len), _i32(budget), ctypes.c_int32(counts.shape[-1]),
                                          new_len, _ptr(workspace),
                                          ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                                          _ptr(status_dev), _stream()))
    return list(new_len)


def kvs_decode_attn_per_head(params: kvs_params_t, q_new, K, V, counts, seq_len: Sequence[int], out,
                             workspace, lse=None, status_dev=None) -> None:
    n_new = q_new.shape[2]
    _check(lib().kvs_decode_attn_per_head(ctypes.byref(params), _ptr(q_new), ctypes.c_int32(n_new), _ptr(K),
                                          _ptr(V), _ptr(counts), _i32(seq_len),
                                          ctypes.c_int32(counts.shape[-1]), _ptr(out), _ptr(lse),
                                          _ptr(workspace),
                                          ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                                          _ptr(status_dev), _stream()))


def kvs_adjacent_cosine(x, seq_len: Sequence[int], cos_out) -> None:
    """cos_out[b,h,t] = cosine of rows t and t+1 of the bf16 tensor x [B,H,Nmax,128], t < seq_len[b]-1."""
    B, H, Nmax, _ = x.shape
    _check(lib().kvs_adjacent_cosine(_ptr(x), ctypes.c_int32(B), ctypes.c_int32(H), ctypes.c_int32(Nmax),
                                     ctypes.c_int64(x.stride(0)), ctypes.c_int64(x.stride(1)),
                                     ctypes.c_int64(x.stride(2)), _i32(seq_len), _ptr(cos_out), _stream()))


def kvs_debug_set_wait(limit_us: int = 0, withhold: int = 0) -> None:
    """Time limit of the device-side waits (0: the default of one second) and the test hook that
    makes one kind of wait run out (see kvs.h)."""
    _check(lib().kvs_debug_set_wait(ctypes.c_uint32(limit_us), ctypes.c_uint32(withhold)))


def kvs_probe_sfu(blocks: int, iters: int, sink) -> int:
    """Launch the special-function probe on the current stream; returns the operations it executes."""
    ops = ctypes.c_uint64(0)
    _check(lib().kvs_probe_sfu(ctypes.c_int32(blocks), ctypes.c_int32(iters), _ptr(sink), ctypes.byref(ops), _stream()))
    return int(ops.value)


def kvs_probe_mma(blocks: int, n_cols: int, reuse_a: bool, products: int, cycles) -> None:
    """Launch the operand-feed probe on the current stream; `cycles` is a device int64[blocks] that
    receives each CTA's elapsed cycles for its `products` tensor-core products (-1: wait ran out)."""
    _check(lib().kvs_probe_mma(ctypes.c_int32(blocks), ctypes.c_int32(n_cols), ctypes.c_int32(1 if reuse_a else 0),
                               ctypes.c_int32(products), _ptr(cycles), _stream()))


def kvs_profile_begin() -> None:
    _check(lib().kvs_profile_begin())


def kvs_profile_end() -> Dict[str, Tuple[float, int]]:
    """{kernel kind: (summed device ms, launches)} since kvs_profile_begin()."""
    names = []
    k = 0
    while True:
        nm = lib().kvs_profile_kind_name(k)
        if nm is None:
            break
        names.append(nm.decode())
        k += 1
    ms = (ctypes.c_float * k)()
    cnt = (ctypes.c_int32 * k)()
    _check(lib().kvs_profile_end(k, ms, cnt))
    return {names[i]: (float(ms[i]), int(cnt[i])) for i in range(k)}
