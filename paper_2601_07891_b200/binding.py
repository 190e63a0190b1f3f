"""ctypes binding of ``libkvzap.so`` (the C ABI declared in ``include/kvzap.h``).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  torch is used for device memory and streams.  There is no CPU
fallback: if the library cannot be loaded, importing a symbol from it raises.

The module-level ``kvzap_*`` functions mirror the C entry points one to one
(tensors instead of raw pointers); :class:`Kvzap` is a small convenience
wrapper that owns a context and allocates outputs.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libkvzap.so")
_lib = None

KVZAP_OK = 0
STATUS_NAMES = {0: "KVZAP_OK", 1: "KVZAP_ERR_INVALID_ARG", 2: "KVZAP_ERR_UNSUPPORTED", 3: "KVZAP_ERR_CUDA",
                4: "KVZAP_ERR_OOM_PAGES", 5: "KVZAP_ERR_TIMEOUT", 6: "KVZAP_ERR_STATE"}


class KvzapError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("%s: %s" % (STATUS_NAMES.get(status, str(status)), message))
        self.status = status


class KvzapConfig(ctypes.Structure):
    _fields_ = [("d_model", ctypes.c_int32), ("hidden", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("n_layers", ctypes.c_int32), ("device", ctypes.c_int32),
                ("max_tokens", ctypes.c_int64), ("max_seqs", ctypes.c_int32), ("flags", ctypes.c_int32)]


_vp, _i32, _i64, _f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float

# name -> (restype, argtypes); also the list of symbols the header declares
SIGNATURES = {
    "kvzap_create": (_i32, [ctypes.POINTER(_vp), ctypes.POINTER(KvzapConfig)]),
    "kvzap_destroy": (_i32, [_vp]),
    "kvzap_last_error": (ctypes.c_char_p, [_vp]),
    "kvzap_set_weights": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _vp]),
    "kvzap_score": (_i32, [_vp, _i32, _vp, _i64, _vp, _vp]),
    "kvzap_prune_prefill": (_i32, [_vp, _vp, _vp, _vp, _vp, _i32, _i64, _f32, _i32, _vp, _vp, _vp, _vp]),
    "kvzap_prefill_fused": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _i32, _i64, _f32, _i32, _vp, _vp, _vp, _vp, _vp]),
    "kvzap_prefill_fused_host": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _i32, _i64, _f32, _i32, _vp, _vp, _vp, _vp,
                                        _vp]),
    "kvzap_prefill_layers_host": (_i32, [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _i32, _i64, _f32, _i32, _vp, _vp, _vp, _vp,
                                         _i32, _i64, _vp, _vp, _i32, _vp, _vp]),
    "kvzap_prefill_fused_paged_host": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _i32, _i64, _f32, _i32, _vp, _vp, _i64, _i32,
                                              _i32, _vp, _i32, _vp, _vp, _vp, _vp]),
    "kvzap_prefill_plan": (_i32, [_vp, _i32, _vp, _vp, _i32, _i64, _f32, _i32, _vp, _vp, _vp, _i32, _i64, _i32, _vp, _i32, _vp,
                                  _vp]),
    "kvzap_set_weights_fp8": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _vp, _vp]),
    "kvzap_score_fp8": (_i32, [_vp, _i32, _vp, _vp, _i64, _vp, _vp]),
    "kvzap_prefill_fused_fp8": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _vp, _i32, _i64, _f32, _i32, _vp, _vp, _vp, _vp, _vp]),
    "kvzap_prune_prefill_noalloc": (_i32, [_vp, _vp, _vp, _vp, _i32, _i64, _i32, _i32, _f32, _i32, _vp, _vp, _vp, _vp]),
    "kvzap_prune_prefill_paged": (_i32, [_vp, _vp, _vp, _vp, _vp, _i32, _i64, _f32, _i32, _vp, _vp, _i64, _i32, _i32,
                                         _vp, _i32, _vp, _vp, _vp]),
    "kvzap_prefill_fused_paged": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _i32, _i64, _f32, _i32, _vp, _vp, _i64, _i32,
                                         _i32, _vp, _i32, _vp, _vp, _vp, _vp]),
    "kvzap_prefill_fused_paged_fp8": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _vp, _i32, _i64, _f32, _i32, _vp, _vp, _i64, _i32,
                                             _i32, _vp, _i32, _vp, _vp, _vp, _vp]),
    "kvzap_prune_prefill_topk": (_i32, [_vp, _vp, _vp, _vp, _vp, _i32, _i64, _f32, _i32, _i32, _vp, _vp, _vp, _vp, _vp]),
    "kvzap_prefill_write": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _i32, _i64, _f32, _i32, _vp, _vp, _vp, _vp, _vp]),
    "kvzap_prefill_write_paged": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _i32, _i64, _f32, _i32, _vp, _vp, _i64, _i32,
                                         _i32, _vp, _i32, _vp, _vp, _vp, _vp]),
    "kvzap_cache_create": (_i32, [_vp, ctypes.POINTER(_vp), _i32, _i32, _i32, _vp, _vp, _i64, _i32]),
    "kvzap_cache_destroy": (_i32, [_vp]),
    "kvzap_decode_step": (_i32, [_vp, _vp, _i32, _i32, _vp, _vp, _vp, _f32, _vp, _vp]),
    "kvzap_decode_step_fp8": (_i32, [_vp, _vp, _i32, _i32, _vp, _vp, _vp, _vp, _f32, _vp, _vp]),
    "kvzap_decode_attention": (_i32, [_vp, _vp, _i32, _i32, _vp, _i32, _f32, _vp, _vp]),
    "kvzap_decode_attention_fp8": (_i32, [_vp, _vp, _i32, _i32, _vp, _i32, _f32, _vp, _vp]),
    "kvzap_cache_release_seq": (_i32, [_vp, _i32, _vp]),
    "kvzap_cache_lengths": (_i32, [_vp, _vp, _vp]),
    "kvzap_cache_export": (_i32, [_vp, _i32, _i32, _i32, _vp, _vp, _i64, _vp, _vp]),
    "kvzap_prefill_to_cache": (_i32, [_vp, _vp, _i32, _i32, _vp, _vp, _vp, _i64, _f32, _vp, _vp]),
    "kvzap_prefill_to_cache_batch": (_i32, [_vp, _vp, _i32, _vp, _vp, _i32, _vp, _vp, _vp, _i64, _f32, _vp, _vp]),
    "kvzap_cache_import": (_i32, [_vp, _vp, _vp, _i32, _vp]),
    "kvzap_cache_snapshot": (_i32, [_vp, _vp, _vp, _vp, _vp]),
    "kvzap_set_wait_limit": (_i32, [_vp, _i64]),
    "kvzap_cache_debug_skew_steps": (_i32, [_vp, _i32]),
    "kvzap_set_profiling": (_i32, [_vp, _i32]),
    "kvzap_get_profile": (_i32, [_vp, _i32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(_i64)]),
    "kvzap_poll_status": (_i32, [_vp, _vp]),
    "kvzap_launch_count": (_i64, [_vp]),
}


def library_path() -> str:
    return _LIB_PATH


def load():
    """Loads libkvzap.so (building it with nvcc first if it is missing or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    try:
        _build.build()
    except Exception as e:  # no nvcc on this machine: fall through to whatever was shipped
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError("libkvzap.so is not built and could not be built here (%s); run "
                               "`python -m paper_2601_07891_b200.build` on a machine with nvcc" % (e,)) from e
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError("libkvzap.so not found at %s" % _LIB_PATH)
    lib = ctypes.CDLL(_LIB_PATH)
    for name, (res, args) in SIGNATURES.items():
        fn = getattr(lib, name)          # AttributeError if the symbol is not exported
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


def _ptr(t):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "tensors must be contiguous CUDA tensors"
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _check(handle, st):
    if st != KVZAP_OK:
        msg = load().kvzap_last_error(handle)
        raise KvzapError(st, msg.decode() if msg else "")


FLAG_TRUSTED_PRODUCERS = 1


def kvzap_create(d_model, hidden, n_kv_heads, head_dim, n_layers, max_tokens, max_seqs=1, device=0, flags=0):
    cfg = KvzapConfig(d_model, hidden, n_kv_heads, head_dim, n_layers, device, max_tokens, max_seqs, flags)
    handle = ctypes.c_void_p()
    st = load().kvzap_create(ctypes.byref(handle), ctypes.byref(cfg))
    _check(None, st)
    return handle


def kvzap_destroy(handle):
    _check(handle, load().kvzap_destroy(handle))


def kvzap_set_weights(handle, layer, W1, b1=None, W2=None, b2=None, stream=None):
    _check(handle, load().kvzap_set_weights(handle, layer, _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), _stream(stream)))


def kvzap_score(handle, layer, hidden, scores, stream=None):
    n_tokens = hidden.shape[0]
    _check(handle, load().kvzap_score(handle, layer, _ptr(hidden) if n_tokens else None, n_tokens,
                                      _ptr(scores) if n_tokens else None, _stream(stream)))


def kvzap_prune_prefill(handle, K, V, scores, cu_seqlens, n_seqs, tau, w, K_out, V_out, lengths, stream=None):
    n_tokens = K.shape[1]
    nz = n_tokens > 0
    _check(handle, load().kvzap_prune_prefill(
        handle, _ptr(K) if nz else None, _ptr(V) if nz else None, _ptr(scores) if nz else None, _ptr(cu_seqlens),
        n_seqs, n_tokens, tau, w, _ptr(K_out) if nz else None, _ptr(V_out) if nz else None, _ptr(lengths),
        _stream(stream)))


def kvzap_prefill_fused(handle, layer, hidden, K, V, cu_seqlens, n_seqs, tau, w, K_out, V_out, lengths,
                        scores_out=None, stream=None):
    n_tokens = K.shape[1]
    nz = n_tokens > 0
    _check(handle, load().kvzap_prefill_fused(
        handle, layer, _ptr(hidden) if nz else None, _ptr(K) if nz else None, _ptr(V) if nz else None,
        _ptr(cu_seqlens), n_seqs, n_tokens, tau, w, _ptr(K_out) if nz else None, _ptr(V_out) if nz else None,
        _ptr(lengths), _ptr(scores_out) if nz else None, _stream(stream)))


def _hptr(t):
    if t is None:
        return None
    assert not t.is_cuda and t.is_contiguous(), "host entry point takes contiguous CPU tensors"
    return ctypes.c_void_p(t.data_ptr())


def kvzap_prefill_fused_host(handle, layer, hidden, K, V, cu_seqlens, n_seqs, tau, w, K_out, V_out, lengths,
                             scores_out=None, stream=None):
    """All tensors are HOST tensors (pinned recommended); returns after the results are on the host."""
    n_tokens = K.shape[1]
    _check(handle, load().kvzap_prefill_fused_host(
        handle, layer, _hptr(hidden), _hptr(K), _hptr(V), _hptr(cu_seqlens), n_seqs, n_tokens, tau, w,
        _hptr(K_out), _hptr(V_out), _hptr(lengths), _hptr(scores_out), _stream(stream)))


def kvzap_prefill_plan(handle, layer, hidden, cu_seqlens, n_seqs, tau, w, slot, lengths, scores_out=None, page_tokens=0,
                       n_pages_pool=0, first_page=0, page_table=None, n_pages_used=None, stream=None):
    """Write plan: slot [n_tokens, H] int32 receives every pair's destination row (-1 = dropped)."""
    n_tokens = hidden.shape[0]
    nz = n_tokens > 0
    _check(handle, load().kvzap_prefill_plan(
        handle, layer, _ptr(hidden) if nz else None, _ptr(cu_seqlens), n_seqs, n_tokens, tau, w, _ptr(slot) if nz else None,
        _ptr(lengths), _ptr(scores_out) if nz else None, page_tokens, n_pages_pool, first_page, _ptr(page_table),
        page_table.shape[1] if page_table is not None else 0, _ptr(n_pages_used), _stream(stream)))


def kvzap_set_weights_fp8(handle, layer, W1_e4m3, w1_scale, b1=None, W2=None, b2=None, stream=None):
    """W1_e4m3: uint8 tensor [rows, d_model] of E4M3 bytes; w1_scale fp32 [rows] or None."""
    _check(handle, load().kvzap_set_weights_fp8(handle, layer, _ptr(W1_e4m3), _ptr(w1_scale), _ptr(b1), _ptr(W2), _ptr(b2),
                                                _stream(stream)))


def kvzap_score_fp8(handle, layer, hidden_e4m3, x_scale, scores, stream=None):
    n_tokens = hidden_e4m3.shape[0]
    _check(handle, load().kvzap_score_fp8(handle, layer, _ptr(hidden_e4m3) if n_tokens else None, _ptr(x_scale), n_tokens,
                                          _ptr(scores) if n_tokens else None, _stream(stream)))


def kvzap_prefill_fused_fp8(handle, layer, hidden_e4m3, x_scale, K, V, cu_seqlens, n_seqs, tau, w, K_out, V_out, lengths,
                            scores_out=None, stream=None):
    n_tokens = K.shape[1]
    nz = n_tokens > 0
    _check(handle, load().kvzap_prefill_fused_fp8(
        handle, layer, _ptr(hidden_e4m3) if nz else None, _ptr(x_scale), _ptr(K) if nz else None, _ptr(V) if nz else None,
        _ptr(cu_seqlens), n_seqs, n_tokens, tau, w, _ptr(K_out) if nz else None, _ptr(V_out) if nz else None,
        _ptr(lengths), _ptr(scores_out) if nz else None, _stream(stream)))


def _hptr_array(tensors):
    """A C array of host pointers (NULL for None entries); returns (array, keep-alive list)."""
    arr = (ctypes.c_void_p * len(tensors))()
    for i, t in enumerate(tensors):
        if t is not None:
            assert not t.is_cuda and t.is_contiguous(), "host entry point takes contiguous CPU tensors"
            arr[i] = t.data_ptr()
    return arr


def kvzap_prefill_layers_host(handle, layer_begin, hidden, K, V, cu_seqlens, n_seqs, tau, w, K_out, V_out, lengths,
                              scores_out=None, page_tokens=0, first_page=None, page_table=None, n_pages_used=None,
                              stream=None):
    """Lists of HOST tensors, one entry per layer of [layer_begin, layer_begin + len(hidden)); paged output when
    page_tokens > 0 (K_out / V_out are then the host pools, first_page a list of ints or None)."""
    n = len(hidden)
    n_tokens = K[0].shape[1]
    args = [_hptr_array(x) for x in (hidden, K, V)]
    outs = [_hptr_array(x) for x in (K_out, V_out, lengths)]
    sc = _hptr_array(scores_out) if scores_out is not None else None
    if page_tokens > 0:
        fp = (ctypes.c_int32 * n)(*(first_page if first_page is not None else [0] * n))
        tab, used = _hptr_array(page_table), _hptr_array(n_pages_used)
        n_pool, max_pages = K_out[0].shape[0], page_table[0].shape[1]
    else:
        fp, tab, used, n_pool, max_pages = None, None, None, 0, 0
    _check(handle, load().kvzap_prefill_layers_host(
        handle, layer_begin, layer_begin + n, args[0], args[1], args[2], _hptr(cu_seqlens), n_seqs, n_tokens, tau, w,
        outs[0], outs[1], outs[2], sc, page_tokens, n_pool, fp, tab, max_pages, used, _stream(stream)))


def kvzap_prefill_fused_paged_host(handle, layer, hidden, K, V, cu_seqlens, n_seqs, tau, w, K_pool, V_pool, page_tokens,
                                   first_page, page_table, lengths, n_pages_used, scores_out=None, stream=None):
    """All tensors are HOST tensors, the pools, the page table and n_pages_used included."""
    _check(handle, load().kvzap_prefill_fused_paged_host(
        handle, layer, _hptr(hidden), _hptr(K), _hptr(V), _hptr(cu_seqlens), n_seqs, K.shape[1], tau, w, _hptr(K_pool),
        _hptr(V_pool), K_pool.shape[0], page_tokens, first_page, _hptr(page_table), page_table.shape[1], _hptr(lengths),
        _hptr(n_pages_used), _hptr(scores_out), _stream(stream)))


NOALLOC_MAX_TOKENS = 131072
NOALLOC_MAX_SEQS = 256


def kvzap_prune_prefill_noalloc(K, V, scores, cu_seqlens, n_seqs, tau, w, K_out, V_out, lengths, stream=None):
    """kvzap_prune_prefill without a context and without any allocation: the scratch is a fixed
    array inside the library (limits NOALLOC_MAX_TOKENS / NOALLOC_MAX_SEQS).  Works on the current
    device; calls that overlap on the GPU race on that array, so keep them on one stream."""
    n_heads, n_tokens, head_dim = K.shape
    nz = n_tokens > 0
    _check(None, load().kvzap_prune_prefill_noalloc(
        _ptr(K) if nz else None, _ptr(V) if nz else None, _ptr(scores) if nz else None, _ptr(cu_seqlens), n_seqs,
        n_tokens, n_heads, head_dim, tau, w, _ptr(K_out) if nz else None, _ptr(V_out) if nz else None,
        _ptr(lengths), _stream(stream)))


def kvzap_prune_prefill_paged(handle, K, V, scores, cu_seqlens, n_seqs, tau, w, K_pool, V_pool, page_tokens,
                              first_page, page_table, lengths, n_pages_used, stream=None):
    n_tokens = K.shape[1]
    nz = n_tokens > 0
    _check(handle, load().kvzap_prune_prefill_paged(
        handle, _ptr(K) if nz else None, _ptr(V) if nz else None, _ptr(scores) if nz else None, _ptr(cu_seqlens),
        n_seqs, n_tokens, tau, w, _ptr(K_pool), _ptr(V_pool), K_pool.shape[0], page_tokens, first_page,
        _ptr(page_table), page_table.shape[1], _ptr(lengths), _ptr(n_pages_used), _stream(stream)))


def kvzap_prefill_fused_paged(handle, layer, hidden, K, V, cu_seqlens, n_seqs, tau, w, K_pool, V_pool, page_tokens,
                              first_page, page_table, lengths, n_pages_used, scores_out=None, stream=None):
    n_tokens = K.shape[1]
    nz = n_tokens > 0
    _check(handle, load().kvzap_prefill_fused_paged(
        handle, layer, _ptr(hidden) if nz else None, _ptr(K) if nz else None, _ptr(V) if nz else None,
        _ptr(cu_seqlens), n_seqs, n_tokens, tau, w, _ptr(K_pool), _ptr(V_pool), K_pool.shape[0], page_tokens,
        first_page, _ptr(page_table), page_table.shape[1], _ptr(lengths), _ptr(n_pages_used),
        _ptr(scores_out) if nz else None, _stream(stream)))


def kvzap_prune_prefill_topk(handle, K, V, scores, cu_seqlens, n_seqs, keep_ratio, w, per_layer, K_out, V_out, lengths,
                             tau_out=None, stream=None):
    n_tokens = K.shape[1]
    nz = n_tokens > 0
    _check(handle, load().kvzap_prune_prefill_topk(
        handle, _ptr(K) if nz else None, _ptr(V) if nz else None, _ptr(scores) if nz else None, _ptr(cu_seqlens),
        n_seqs, n_tokens, keep_ratio, w, 1 if per_layer else 0, _ptr(K_out) if nz else None, _ptr(V_out) if nz else None,
        _ptr(lengths), _ptr(tau_out), _stream(stream)))


def kvzap_prefill_write(handle, layer, hidden, K_proj, V_proj, cu_seqlens, n_seqs, tau, w, K_out, V_out, lengths,
                        scores_out=None, stream=None):
    """K_proj, V_proj [n_tokens, H, D]: the projection's own layout."""
    n_tokens = K_proj.shape[0]
    nz = n_tokens > 0
    _check(handle, load().kvzap_prefill_write(
        handle, layer, _ptr(hidden) if nz else None, _ptr(K_proj) if nz else None, _ptr(V_proj) if nz else None,
        _ptr(cu_seqlens), n_seqs, n_tokens, tau, w, _ptr(K_out) if nz else None, _ptr(V_out) if nz else None,
        _ptr(lengths), _ptr(scores_out) if nz else None, _stream(stream)))


def kvzap_prefill_write_paged(handle, layer, hidden, K_proj, V_proj, cu_seqlens, n_seqs, tau, w, K_pool, V_pool,
                              page_tokens, first_page, page_table, lengths, n_pages_used, scores_out=None, stream=None):
    n_tokens = K_proj.shape[0]
    nz = n_tokens > 0
    _check(handle, load().kvzap_prefill_write_paged(
        handle, layer, _ptr(hidden) if nz else None, _ptr(K_proj) if nz else None, _ptr(V_proj) if nz else None,
        _ptr(cu_seqlens), n_seqs, n_tokens, tau, w, _ptr(K_pool), _ptr(V_pool), K_pool.shape[0], page_tokens,
        first_page, _ptr(page_table), page_table.shape[1], _ptr(lengths), _ptr(n_pages_used),
        _ptr(scores_out) if nz else None, _stream(stream)))


def kvzap_cache_create(handle, n_seqs, window, page_tokens, K_pool, V_pool, max_pages_per_list):
    cache = ctypes.c_void_p()
    _check(handle, load().kvzap_cache_create(handle, ctypes.byref(cache), n_seqs, window, page_tokens, _ptr(K_pool),
                                             _ptr(V_pool), K_pool.shape[0], max_pages_per_list))
    return cache


def kvzap_cache_destroy(cache):
    _check(None, load().kvzap_cache_destroy(cache))


def kvzap_decode_step(handle, cache, layer_begin, layer_end, hidden, K_new, V_new, tau, scores_out=None, stream=None):
    _check(handle, load().kvzap_decode_step(handle, cache, layer_begin, layer_end, _ptr(hidden), _ptr(K_new),
                                            _ptr(V_new), tau, _ptr(scores_out), _stream(stream)))


def kvzap_decode_step_fp8(handle, cache, layer_begin, layer_end, hidden_e4m3, x_scale, K_new, V_new, tau, scores_out=None,
                          stream=None):
    """hidden_e4m3: uint8 [layers, n_seqs, d_model] of E4M3 bytes; x_scale fp32 [layers, n_seqs] or None."""
    _check(handle, load().kvzap_decode_step_fp8(handle, cache, layer_begin, layer_end, _ptr(hidden_e4m3), _ptr(x_scale),
                                                _ptr(K_new), _ptr(V_new), tau, _ptr(scores_out), _stream(stream)))


def kvzap_cache_release_seq(handle, cache, seq, stream=None):
    _check(handle, load().kvzap_cache_release_seq(cache, seq, _stream(stream)))


def kvzap_cache_lengths(handle, cache, lengths, stream=None):
    _check(handle, load().kvzap_cache_lengths(cache, _ptr(lengths), _stream(stream)))


def kvzap_cache_export(handle, cache, seq, layer, head, K_out, V_out, n_rows, stream=None):
    _check(handle, load().kvzap_cache_export(cache, seq, layer, head, _ptr(K_out), _ptr(V_out), K_out.shape[0],
                                             _ptr(n_rows), _stream(stream)))


def kvzap_prefill_to_cache(handle, cache, layer, seq, hidden, K, V, tau, scores_out, stream=None):
    _check(handle, load().kvzap_prefill_to_cache(handle, cache, layer, seq, _ptr(hidden), _ptr(K), _ptr(V), K.shape[1],
                                                 tau, _ptr(scores_out), _stream(stream)))


def kvzap_prefill_to_cache_batch(handle, cache, layer, seq_ids, cu_seqlens, hidden, K, V, tau, scores_out, stream=None):
    """seq_ids: a Python sequence of slot numbers (host); cu_seqlens int32 [len(seq_ids) + 1] on the device;
    hidden [n_tokens, d_model], K, V [H, n_tokens, D] packed over the sequences."""
    ids = (ctypes.c_int32 * len(seq_ids))(*[int(x) for x in seq_ids])
    _check(handle, load().kvzap_prefill_to_cache_batch(handle, cache, layer, ctypes.cast(ids, ctypes.c_void_p), _ptr(cu_seqlens),
                                                       len(seq_ids), _ptr(hidden), _ptr(K), _ptr(V), K.shape[1], tau,
                                                       _ptr(scores_out), _stream(stream)))


def kvzap_cache_import(handle, cache, prefix_len, page_table, next_free_page, stream=None):
    _check(handle, load().kvzap_cache_import(cache, _ptr(prefix_len), _ptr(page_table), next_free_page,
                                             _stream(stream)))


def kvzap_cache_snapshot(handle, cache, prefix_len, page_table, next_free_page, stream=None):
    _check(handle, load().kvzap_cache_snapshot(cache, _ptr(prefix_len), _ptr(page_table), _ptr(next_free_page),
                                               _stream(stream)))


class PreparedCall:
    """One C entry point with its arguments marshalled once.  For loops that repeat the same call on the
    same buffers (a benchmark step, a serving loop with fixed buffers): calling it costs one ctypes
    call instead of re-wrapping a dozen tensors.  The tensors are kept alive by the object; the
    stream is the one current when it was prepared (or the one given)."""

    __slots__ = ("_fn", "_args", "_handle", "_keep")

    def __init__(self, name, handle, args, keep):
        self._fn = getattr(load(), name)
        self._args = args
        self._handle = handle
        self._keep = keep

    def __call__(self):
        st = self._fn(*self._args)
        if st != KVZAP_OK:
            _check(self._handle, st)


def prepare_prefill_fused(handle, layer, hidden, K, V, cu_seqlens, n_seqs, tau, w, K_out, V_out, lengths,
                          scores_out=None, stream=None) -> PreparedCall:
    """kvzap_prefill_fused with pre-marshalled arguments (see PreparedCall)."""
    args = (handle, layer, _ptr(hidden), _ptr(K), _ptr(V), _ptr(cu_seqlens), n_seqs, K.shape[1], tau, w, _ptr(K_out),
            _ptr(V_out), _ptr(lengths), _ptr(scores_out), _stream(stream))
    return PreparedCall("kvzap_prefill_fused", handle, args, (hidden, K, V, cu_seqlens, K_out, V_out, lengths, scores_out))


def prepare_prune_prefill(handle, K, V, scores, cu_seqlens, n_seqs, tau, w, K_out, V_out, lengths, stream=None) -> PreparedCall:
    args = (handle, _ptr(K), _ptr(V), _ptr(scores), _ptr(cu_seqlens), n_seqs, K.shape[1], tau, w, _ptr(K_out), _ptr(V_out),
            _ptr(lengths), _stream(stream))
    return PreparedCall("kvzap_prune_prefill", handle, args, (K, V, scores, cu_seqlens, K_out, V_out, lengths))


def prepare_prune_prefill_paged(handle, K, V, scores, cu_seqlens, n_seqs, tau, w, K_pool, V_pool, page_tokens, first_page,
                                page_table, lengths, n_pages_used, stream=None) -> PreparedCall:
    args = (handle, _ptr(K), _ptr(V), _ptr(scores), _ptr(cu_seqlens), n_seqs, K.shape[1], tau, w, _ptr(K_pool), _ptr(V_pool),
            K_pool.shape[0], page_tokens, first_page, _ptr(page_table), page_table.shape[1], _ptr(lengths),
            _ptr(n_pages_used), _stream(stream))
    return PreparedCall("kvzap_prune_prefill_paged", handle, args,
                        (K, V, scores, cu_seqlens, K_pool, V_pool, page_table, lengths, n_pages_used))


def prepare_prefill_fused_fp8(handle, layer, hidden_e4m3, x_scale, K, V, cu_seqlens, n_seqs, tau, w, K_out, V_out, lengths,
                              scores_out=None, stream=None) -> PreparedCall:
    args = (handle, layer, _ptr(hidden_e4m3), _ptr(x_scale), _ptr(K), _ptr(V), _ptr(cu_seqlens), n_seqs, K.shape[1], tau, w,
            _ptr(K_out), _ptr(V_out), _ptr(lengths), _ptr(scores_out), _stream(stream))
    return PreparedCall("kvzap_prefill_fused_fp8", handle, args,
                        (hidden_e4m3, x_scale, K, V, cu_seqlens, K_out, V_out, lengths, scores_out))


def _paged_fp8_args(handle, layer, hidden_e4m3, x_scale, K, V, cu_seqlens, n_seqs, tau, w, K_pool, V_pool, page_tokens,
                    first_page, page_table, lengths, n_pages_used, scores_out, stream):
    return (handle, layer, _ptr(hidden_e4m3), _ptr(x_scale), _ptr(K), _ptr(V), _ptr(cu_seqlens), n_seqs, K.shape[1], tau, w,
            _ptr(K_pool), _ptr(V_pool), K_pool.shape[0], page_tokens, first_page, _ptr(page_table), page_table.shape[1],
            _ptr(lengths), _ptr(n_pages_used), _ptr(scores_out), _stream(stream))


def kvzap_prefill_fused_paged_fp8(handle, layer, hidden_e4m3, x_scale, K, V, cu_seqlens, n_seqs, tau, w, K_pool, V_pool,
                                  page_tokens, first_page, page_table, lengths, n_pages_used, scores_out=None, stream=None):
    """kvzap_prefill_fused_paged with hidden states as E4M3 bytes [n_tokens, d_model] and x_scale fp32 [n_tokens] or None."""
    _check(handle, load().kvzap_prefill_fused_paged_fp8(*_paged_fp8_args(
        handle, layer, hidden_e4m3, x_scale, K, V, cu_seqlens, n_seqs, tau, w, K_pool, V_pool, page_tokens, first_page,
        page_table, lengths, n_pages_used, scores_out, stream)))


def prepare_prefill_fused_paged_fp8(handle, layer, hidden_e4m3, x_scale, K, V, cu_seqlens, n_seqs, tau, w, K_pool, V_pool,
                                    page_tokens, first_page, page_table, lengths, n_pages_used, scores_out=None,
                                    stream=None) -> PreparedCall:
    args = _paged_fp8_args(handle, layer, hidden_e4m3, x_scale, K, V, cu_seqlens, n_seqs, tau, w, K_pool, V_pool, page_tokens,
                           first_page, page_table, lengths, n_pages_used, scores_out, stream)
    return PreparedCall("kvzap_prefill_fused_paged_fp8", handle, args,
                        (hidden_e4m3, x_scale, K, V, cu_seqlens, K_pool, V_pool, page_table, lengths, n_pages_used, scores_out))


def prepare_prefill_fused_paged(handle, layer, hidden, K, V, cu_seqlens, n_seqs, tau, w, K_pool, V_pool, page_tokens,
                                first_page, page_table, lengths, n_pages_used, scores_out=None, stream=None) -> PreparedCall:
    args = (handle, layer, _ptr(hidden), _ptr(K), _ptr(V), _ptr(cu_seqlens), n_seqs, K.shape[1], tau, w, _ptr(K_pool),
            _ptr(V_pool), K_pool.shape[0], page_tokens, first_page, _ptr(page_table), page_table.shape[1], _ptr(lengths),
            _ptr(n_pages_used), _ptr(scores_out), _stream(stream))
    return PreparedCall("kvzap_prefill_fused_paged", handle, args,
                        (hidden, K, V, cu_seqlens, K_pool, V_pool, page_table, lengths, n_pages_used, scores_out))


def prepare_prefill_write(handle, layer, hidden, K_proj, V_proj, cu_seqlens, n_seqs, tau, w, K_out, V_out, lengths,
                          scores_out=None, stream=None) -> PreparedCall:
    args = (handle, layer, _ptr(hidden), _ptr(K_proj), _ptr(V_proj), _ptr(cu_seqlens), n_seqs, K_proj.shape[0], tau, w,
            _ptr(K_out), _ptr(V_out), _ptr(lengths), _ptr(scores_out), _stream(stream))
    return PreparedCall("kvzap_prefill_write", handle, args,
                        (hidden, K_proj, V_proj, cu_seqlens, K_out, V_out, lengths, scores_out))


def prepare_prefill_write_paged(handle, layer, hidden, K_proj, V_proj, cu_seqlens, n_seqs, tau, w, K_pool, V_pool,
                                page_tokens, first_page, page_table, lengths, n_pages_used, scores_out=None,
                                stream=None) -> PreparedCall:
    args = (handle, layer, _ptr(hidden), _ptr(K_proj), _ptr(V_proj), _ptr(cu_seqlens), n_seqs, K_proj.shape[0], tau, w,
            _ptr(K_pool), _ptr(V_pool), K_pool.shape[0], page_tokens, first_page, _ptr(page_table), page_table.shape[1],
            _ptr(lengths), _ptr(n_pages_used), _ptr(scores_out), _stream(stream))
    return PreparedCall("kvzap_prefill_write_paged", handle, args,
                        (hidden, K_proj, V_proj, cu_seqlens, K_pool, V_pool, page_table, lengths, n_pages_used, scores_out))


def kvzap_decode_attention(handle, cache, layer_begin, layer_end, Q, scale, O, stream=None):
    """Q, O [layer_end - layer_begin, n_seqs, n_q_heads, D] bf16 on the device."""
    _check(handle, load().kvzap_decode_attention(handle, cache, layer_begin, layer_end, _ptr(Q), Q.shape[2], scale,
                                                 _ptr(O), _stream(stream)))


def prepare_decode_attention(handle, cache, layer_begin, layer_end, Q, scale, O, stream=None) -> PreparedCall:
    args = (handle, cache, layer_begin, layer_end, _ptr(Q), Q.shape[2], scale, _ptr(O), _stream(stream))
    return PreparedCall("kvzap_decode_attention", handle, args, (Q, O))


def kvzap_decode_attention_fp8(handle, cache, layer_begin, layer_end, Q, scale, O, stream=None):
    """Cache rows are E4M3 codes + a 16-byte trailer (fp32 scale first); Q, O [layers, n_seqs, n_q_heads, D] bf16."""
    _check(handle, load().kvzap_decode_attention_fp8(handle, cache, layer_begin, layer_end, _ptr(Q), Q.shape[2], scale,
                                                     _ptr(O), _stream(stream)))


def prepare_decode_attention_fp8(handle, cache, layer_begin, layer_end, Q, scale, O, stream=None) -> PreparedCall:
    args = (handle, cache, layer_begin, layer_end, _ptr(Q), Q.shape[2], scale, _ptr(O), _stream(stream))
    return PreparedCall("kvzap_decode_attention_fp8", handle, args, (Q, O))


def prepare_decode_step(handle, cache, layer_begin, layer_end, hidden, K_new, V_new, tau, scores_out=None,
                        stream=None) -> PreparedCall:
    args = (handle, cache, layer_begin, layer_end, _ptr(hidden), _ptr(K_new), _ptr(V_new), tau, _ptr(scores_out),
            _stream(stream))
    return PreparedCall("kvzap_decode_step", handle, args, (hidden, K_new, V_new, scores_out))


def prepare_decode_step_fp8(handle, cache, layer_begin, layer_end, hidden_e4m3, x_scale, K_new, V_new, tau, scores_out=None,
                            stream=None) -> PreparedCall:
    args = (handle, cache, layer_begin, layer_end, _ptr(hidden_e4m3), _ptr(x_scale), _ptr(K_new), _ptr(V_new), tau,
            _ptr(scores_out), _stream(stream))
    return PreparedCall("kvzap_decode_step_fp8", handle, args, (hidden_e4m3, x_scale, K_new, V_new, scores_out))


KERNEL_IDS = {"score": 0, "mask": 1, "scan": 2, "compact": 3, "decode_update": 4, "attention": 5}


def kvzap_set_profiling(handle, enable):
    _check(handle, load().kvzap_set_profiling(handle, 1 if enable else 0))


def kvzap_get_profile(handle, kernel):
    """-> (total_ms, n_launches) of one kernel since profiling was switched on."""
    ms, n = ctypes.c_double(0.0), ctypes.c_int64(0)
    _check(handle, load().kvzap_get_profile(handle, KERNEL_IDS[kernel] if isinstance(kernel, str) else kernel,
                                            ctypes.byref(ms), ctypes.byref(n)))
    return float(ms.value), int(n.value)


def kvzap_set_wait_limit(handle, cycles):
    _check(handle, load().kvzap_set_wait_limit(handle, cycles))


def kvzap_cache_debug_skew_steps(cache, delta):
    """Test aid: makes the next fused decode step wait for a step that never ran (see the header)."""
    _check(None, load().kvzap_cache_debug_skew_steps(cache, delta))


def kvzap_poll_status(handle, stream=None) -> int:
    return int(load().kvzap_poll_status(handle, _stream(stream)))


def kvzap_launch_count(handle) -> int:
    return int(load().kvzap_launch_count(handle))


class Kvzap:
    """Owns one context; allocates outputs with torch; same calls as the C ABI."""

    def __init__(self, d_model, hidden, n_kv_heads, head_dim, n_layers, max_tokens, max_seqs=1, device=0,
                 trusted_producers=False):
        """trusted_producers: the caller vouches that the inputs of every call are complete before the
        previous call on the stream was enqueued (KVZAP_FLAG_TRUSTED_PRODUCERS): full overlap of
        consecutive calls.  Off, a call's first kernel waits for the work ahead of it in the stream."""
        self.d_model, self.hidden, self.n_kv_heads, self.head_dim = d_model, hidden, n_kv_heads, head_dim
        self.n_layers, self.max_tokens, self.max_seqs = n_layers, max_tokens, max_seqs
        self.device = torch.device("cuda", device)
        self.handle = kvzap_create(d_model, hidden, n_kv_heads, head_dim, n_layers, max_tokens, max_seqs, device,
                                   FLAG_TRUSTED_PRODUCERS if trusted_producers else 0)

    def close(self):
        if self.handle is not None:
            kvzap_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_weights(self, layer, *weights, stream=None):
        """weights = (W, b) for KVzap-Linear or (W1, b1, W2, b2) for KVzap-MLP."""
        if len(weights) == 2:
            kvzap_set_weights(self.handle, layer, weights[0], weights[1], None, None, stream)
        else:
            kvzap_set_weights(self.handle, layer, *weights, stream=stream)

    def score(self, layer, hidden, out=None, stream=None):
        if hidden.dim() != 2 or hidden.shape[1] != self.d_model or hidden.dtype != torch.bfloat16:
            raise ValueError("hidden must be bf16 [T, %d], got %s" % (self.d_model, tuple(hidden.shape)))
        if out is None:
            out = torch.empty(hidden.shape[0], self.n_kv_heads, dtype=torch.float32, device=self.device)
        kvzap_score(self.handle, layer, hidden, out, stream)
        return out

    def _check_shapes(self, K, V, hidden=None, scores=None):
        """Shape errors are raised here, on the host: the C ABI takes raw pointers and trusts them."""
        if tuple(K.shape[::2]) != (self.n_kv_heads, self.head_dim) or K.shape != V.shape or K.dtype != torch.bfloat16:
            raise ValueError("K/V must be bf16 [%d, T, %d], got %s / %s" % (self.n_kv_heads, self.head_dim,
                                                                            tuple(K.shape), tuple(V.shape)))
        if hidden is not None and (hidden.shape != (K.shape[1], self.d_model) or hidden.dtype != torch.bfloat16):
            raise ValueError("hidden must be bf16 [%d, %d], got %s" % (K.shape[1], self.d_model, tuple(hidden.shape)))
        if scores is not None and (scores.shape != (K.shape[1], self.n_kv_heads) or scores.dtype != torch.float32):
            raise ValueError("scores must be fp32 [%d, %d], got %s" % (K.shape[1], self.n_kv_heads, tuple(scores.shape)))

    def _outputs(self, K, n_seqs, K_out, V_out, lengths):
        if K_out is None:
            K_out = torch.empty_like(K)
        if V_out is None:
            V_out = torch.empty_like(K)
        if lengths is None:
            lengths = torch.empty(n_seqs, self.n_kv_heads, dtype=torch.int32, device=self.device)
        return K_out, V_out, lengths

    def prune_prefill(self, K, V, scores, tau, w, cu_seqlens=None, K_out=None, V_out=None, lengths=None, stream=None):
        n_seqs = 1 if cu_seqlens is None else cu_seqlens.numel() - 1
        self._check_shapes(K, V, scores=scores)
        K_out, V_out, lengths = self._outputs(K, n_seqs, K_out, V_out, lengths)
        kvzap_prune_prefill(self.handle, K, V, scores, cu_seqlens, n_seqs, tau, w, K_out, V_out, lengths, stream)
        return K_out, V_out, lengths

    def prefill_fused(self, layer, hidden, K, V, tau, w, cu_seqlens=None, K_out=None, V_out=None, lengths=None,
                      scores_out=None, stream=None):
        n_seqs = 1 if cu_seqlens is None else cu_seqlens.numel() - 1
        self._check_shapes(K, V, hidden=hidden, scores=scores_out)
        K_out, V_out, lengths = self._outputs(K, n_seqs, K_out, V_out, lengths)
        kvzap_prefill_fused(self.handle, layer, hidden, K, V, cu_seqlens, n_seqs, tau, w, K_out, V_out, lengths,
                            scores_out, stream)
        return K_out, V_out, lengths

    def prefill_write(self, layer, hidden, K_proj, V_proj, tau, w, cu_seqlens=None, K_out=None, V_out=None, lengths=None,
                      scores_out=None, stream=None):
        """Write-side pruning: K_proj, V_proj [T, H, D] as the projection leaves them -> per-head lists [H, T, D]."""
        n_seqs = 1 if cu_seqlens is None else cu_seqlens.numel() - 1
        T = K_proj.shape[0]
        if tuple(K_proj.shape[1:]) != (self.n_kv_heads, self.head_dim) or K_proj.shape != V_proj.shape or \
                K_proj.dtype != torch.bfloat16:
            raise ValueError("K_proj/V_proj must be bf16 [T, %d, %d]" % (self.n_kv_heads, self.head_dim))
        if hidden.shape != (T, self.d_model) or hidden.dtype != torch.bfloat16:
            raise ValueError("hidden must be bf16 [%d, %d], got %s" % (T, self.d_model, tuple(hidden.shape)))
        if K_out is None:
            K_out = torch.empty(self.n_kv_heads, T, self.head_dim, dtype=torch.bfloat16, device=self.device)
        if V_out is None:
            V_out = torch.empty_like(K_out)
        if lengths is None:
            lengths = torch.empty(n_seqs, self.n_kv_heads, dtype=torch.int32, device=self.device)
        kvzap_prefill_write(self.handle, layer, hidden, K_proj, V_proj, cu_seqlens, n_seqs, tau, w, K_out, V_out, lengths,
                            scores_out, stream)
        return K_out, V_out, lengths

    def prune_prefill_topk(self, K, V, scores, keep_ratio, w, per_layer=False, cu_seqlens=None, K_out=None, V_out=None,
                           lengths=None, tau_out=None, stream=None):
        """Fixed-budget selection (top-k per head, or per layer) instead of a threshold."""
        n_seqs = 1 if cu_seqlens is None else cu_seqlens.numel() - 1
        self._check_shapes(K, V, scores=scores)
        K_out, V_out, lengths = self._outputs(K, n_seqs, K_out, V_out, lengths)
        kvzap_prune_prefill_topk(self.handle, K, V, scores, cu_seqlens, n_seqs, keep_ratio, w, per_layer, K_out, V_out,
                                 lengths, tau_out, stream)
        return K_out, V_out, lengths

    def create_cache(self, n_seqs, window, page_tokens, K_pool, V_pool, max_pages_per_list) -> "KvzapCache":
        return KvzapCache(self, n_seqs, window, page_tokens, K_pool, V_pool, max_pages_per_list)

    def poll_status(self, stream=None) -> int:
        return kvzap_poll_status(self.handle, stream)

    def launch_count(self) -> int:
        return kvzap_launch_count(self.handle)


class KvzapCache:
    """The decode-time cache of one context (window ring + paged prefix per (sequence, layer, head) list).
    The page pools stay the caller's tensors; the object keeps them alive."""

    def __init__(self, ctx: Kvzap, n_seqs, window, page_tokens, K_pool, V_pool, max_pages_per_list):
        self.ctx, self.n_seqs, self.window, self.page_tokens = ctx, n_seqs, window, page_tokens
        self._pools = (K_pool, V_pool)
        self.handle = kvzap_cache_create(ctx.handle, n_seqs, window, page_tokens, K_pool, V_pool, max_pages_per_list)

    def close(self):
        if self.handle is not None:
            kvzap_cache_destroy(self.handle)
            self.handle = None

    def prefill(self, layer, seq, hidden, K, V, tau, scores_out=None, stream=None):
        """One prompt, or the next chunk of it, for one layer (chunks of any lengths give the same lists)."""
        if scores_out is None:
            scores_out = torch.empty(K.shape[1], self.ctx.n_kv_heads, dtype=torch.float32, device=self.ctx.device)
        kvzap_prefill_to_cache(self.ctx.handle, self.handle, layer, seq, hidden, K, V, tau, scores_out, stream)
        return scores_out

    def decode_step(self, layer_begin, layer_end, hidden, K_new, V_new, tau, scores_out=None, stream=None):
        kvzap_decode_step(self.ctx.handle, self.handle, layer_begin, layer_end, hidden, K_new, V_new, tau, scores_out, stream)

    def attention(self, layer_begin, layer_end, Q, scale=None, out=None, stream=None):
        """The newest token's attention over the pruned lists: Q [L, B, H_q, D] -> O of the same shape."""
        if out is None:
            out = torch.empty_like(Q)
        if scale is None:
            scale = 1.0 / float(self.ctx.head_dim) ** 0.5
        kvzap_decode_attention(self.ctx.handle, self.handle, layer_begin, layer_end, Q, scale, out, stream)
        return out

    def release_seq(self, seq, stream=None):
        """The sequence in slot `seq` has ended: its lists become empty and its pages are handed out again."""
        kvzap_cache_release_seq(self.ctx.handle, self.handle, seq, stream)

    def lengths(self, stream=None):
        out = torch.empty(self.n_seqs, self.ctx.n_layers, self.ctx.n_kv_heads, dtype=torch.int32, device=self.ctx.device)
        kvzap_cache_lengths(self.ctx.handle, self.handle, out, stream)
        return out
