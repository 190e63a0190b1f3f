"""ctypes front end of the KVzap CPU oracle -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's cpu_baseline / reference
legs may import this module; the CUDA library never does.  It wraps
``kvzap_oracle.c`` (compiled to ``libkvzap_oracle.so`` beside it) and adds the
decode-time oracle, which follows the caption of Algorithm 1: decoding applies
the same rule as prefilling with a buffer of the scores of the tokens that
are still inside the sliding window.

bf16 tensors are numpy ``uint16`` arrays of raw bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from collections import deque

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kvzap_oracle.c")
_LIB = os.path.join(_HERE, "libkvzap_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C + OpenMP); returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", tmp, _SRC, "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _c(arr, ctype):
    return arr.ctypes.data_as(ctypes.POINTER(ctype)) if arr is not None else None


def lib():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        L.kvzap_oracle_num_threads.restype = ctypes.c_int
        L.kvzap_oracle_gelu.restype = ctypes.c_double
        L.kvzap_oracle_gelu.argtypes = [ctypes.c_double]
        L.kvzap_oracle_score_mlp.restype = ctypes.c_int
        L.kvzap_oracle_compact_paged.restype = ctypes.c_int
        L.kvzap_oracle_compact_write_paged.restype = ctypes.c_int
        L.kvzap_oracle_attention.restype = ctypes.c_int
        L.kvzap_oracle_topk_mask.restype = ctypes.c_int
        for name in ("layer_flops", "mlp_flops", "linear_flops"):
            getattr(L, "kvzap_oracle_" + name).restype = ctypes.c_double
        L.kvzap_oracle_layer_flops.argtypes = [ctypes.c_int] * 5
        L.kvzap_oracle_mlp_flops.argtypes = [ctypes.c_int] * 3
        L.kvzap_oracle_linear_flops.argtypes = [ctypes.c_int] * 2
        L.kvzap_oracle_plan.restype = ctypes.c_int
        L.kvzap_oracle_e4m3_to_double.restype = ctypes.c_double
        L.kvzap_oracle_e4m3_to_double.argtypes = [ctypes.c_uint8]
        L.kvzap_oracle_score_mlp_fp8.restype = ctypes.c_int
        L.kvzap_oracle_attention_fp8.restype = ctypes.c_int
        L.kvzap_oracle_param_count.restype = ctypes.c_int64
        L.kvzap_oracle_param_count.argtypes = [ctypes.c_int] * 3
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().kvzap_oracle_num_threads())


def _u16(a, shape_len):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16 and a.ndim == shape_len, (a.dtype, a.shape)
    return a


def _f32_or_none(a, n):
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype=np.float32)
    assert a.shape == (n,)
    return a


def gelu(x: float) -> float:
    return float(lib().kvzap_oracle_gelu(float(x)))


def score_linear(X, W, b=None):
    """X [T,Dh] bf16 bits, W [H,Dh] bf16 bits, b [H] fp32|None -> scores [T,H] fp32."""
    X = _u16(X, 2)
    W = _u16(W, 2)
    T, Dh = X.shape
    H = W.shape[0]
    assert W.shape[1] == Dh
    b = _f32_or_none(b, H)
    out = np.empty((T, H), dtype=np.float32)
    lib().kvzap_oracle_score_linear(
        _c(X, ctypes.c_uint16), ctypes.c_int64(T), ctypes.c_int(Dh),
        _c(W, ctypes.c_uint16), _c(b, ctypes.c_float), ctypes.c_int(H), _c(out, ctypes.c_float))
    return out


def score_mlp(X, W1, b1, W2, b2):
    """X [T,Dh], W1 [N1,Dh], W2 [H,N1] bf16 bits; b1 [N1], b2 [H] fp32|None -> [T,H] fp32."""
    X = _u16(X, 2)
    W1 = _u16(W1, 2)
    W2 = _u16(W2, 2)
    T, Dh = X.shape
    N1 = W1.shape[0]
    H = W2.shape[0]
    assert W1.shape[1] == Dh and W2.shape[1] == N1
    b1 = _f32_or_none(b1, N1)
    b2 = _f32_or_none(b2, H)
    out = np.empty((T, H), dtype=np.float32)
    rc = lib().kvzap_oracle_score_mlp(
        _c(X, ctypes.c_uint16), ctypes.c_int64(T), ctypes.c_int(Dh),
        _c(W1, ctypes.c_uint16), _c(b1, ctypes.c_float), ctypes.c_int(N1),
        _c(W2, ctypes.c_uint16), _c(b2, ctypes.c_float), ctypes.c_int(H), _c(out, ctypes.c_float))
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return out


def score(X, weights):
    """weights = (W, b) for KVzap-Linear or (W1, b1, W2, b2) for KVzap-MLP."""
    if len(weights) == 2:
        return score_linear(X, *weights)
    return score_mlp(X, *weights)


def _cu(cu_seqlens, T_total):
    if cu_seqlens is None:
        cu_seqlens = [0, T_total]
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    assert cu.ndim == 1 and cu[0] == 0 and cu[-1] == T_total and np.all(np.diff(cu) >= 0)
    return cu


def keep_mask(scores, tau, w, cu_seqlens=None):
    """scores [T_total,H] fp32 -> keep [H,T_total] uint8 (window per sequence)."""
    scores = np.ascontiguousarray(scores, dtype=np.float32)
    T_total, H = scores.shape
    assert w >= 0
    cu = _cu(cu_seqlens, T_total)
    keep = np.zeros((H, T_total), dtype=np.uint8)
    lib().kvzap_oracle_keep_mask(
        _c(scores, ctypes.c_float), _c(cu, ctypes.c_int32), ctypes.c_int(len(cu) - 1),
        ctypes.c_int(H), ctypes.c_float(tau), ctypes.c_int(w), _c(keep, ctypes.c_uint8))
    return keep


def topk_mask(scores, keep_ratio, w, per_layer=False, cu_seqlens=None):
    """Fixed-budget selection: scores [T_total,H] fp32 -> (keep [H,T_total] uint8, tau [B,H] fp32)."""
    scores = np.ascontiguousarray(scores, dtype=np.float32)
    T_total, H = scores.shape
    assert w >= 0
    cu = _cu(cu_seqlens, T_total)
    B = len(cu) - 1
    keep = np.zeros((H, T_total), dtype=np.uint8)
    tau = np.zeros((B, H), dtype=np.float32)
    rc = lib().kvzap_oracle_topk_mask(
        _c(scores, ctypes.c_float), _c(cu, ctypes.c_int32), ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(w),
        ctypes.c_double(float(np.float32(keep_ratio))), ctypes.c_int(1 if per_layer else 0),
        _c(keep, ctypes.c_uint8), _c(tau, ctypes.c_float))
    if rc != 0:
        raise MemoryError("oracle top-k: out of memory")
    return keep, tau


def compact(K, V, keep, cu_seqlens=None, fill=0):
    """K,V [H,T_total,D] bf16 bits, keep [H,T_total] -> (K_out, V_out, lengths[B,H]).

    Outputs are pre-filled with ``fill`` so that untouched rows are visible."""
    K = _u16(K, 3)
    V = _u16(V, 3)
    H, T_total, D = K.shape
    assert V.shape == K.shape
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    assert keep.shape == (H, T_total)
    cu = _cu(cu_seqlens, T_total)
    B = len(cu) - 1
    K_out = np.full_like(K, fill)
    V_out = np.full_like(V, fill)
    lengths = np.zeros((B, H), dtype=np.int32)
    lib().kvzap_oracle_compact(
        _c(K, ctypes.c_uint16), _c(V, ctypes.c_uint16), _c(keep, ctypes.c_uint8),
        _c(cu, ctypes.c_int32), ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(D),
        _c(K_out, ctypes.c_uint16), _c(V_out, ctypes.c_uint16), _c(lengths, ctypes.c_int32))
    return K_out, V_out, lengths


def compact_paged(K, V, keep, page_tokens, n_pages_pool, max_pages_per_list,
                  cu_seqlens=None, first_page=0, fill=0):
    """Paged compaction -> (K_pool, V_pool, page_table[B*H,max_pages], lengths[B,H], n_pages_used).

    page_table entries that are not assigned keep the value -1."""
    K = _u16(K, 3)
    V = _u16(V, 3)
    H, T_total, D = K.shape
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    cu = _cu(cu_seqlens, T_total)
    B = len(cu) - 1
    K_pool = np.full((n_pages_pool, page_tokens, D), fill, dtype=np.uint16)
    V_pool = np.full((n_pages_pool, page_tokens, D), fill, dtype=np.uint16)
    table = np.full((B * H, max_pages_per_list), -1, dtype=np.int32)
    lengths = np.zeros((B, H), dtype=np.int32)
    used = ctypes.c_int32(0)
    rc = lib().kvzap_oracle_compact_paged(
        _c(K, ctypes.c_uint16), _c(V, ctypes.c_uint16), _c(keep, ctypes.c_uint8),
        _c(cu, ctypes.c_int32), ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(D),
        ctypes.c_int(page_tokens), ctypes.c_int32(first_page), ctypes.c_int64(n_pages_pool),
        ctypes.c_int(max_pages_per_list),
        _c(K_pool, ctypes.c_uint16), _c(V_pool, ctypes.c_uint16), _c(table, ctypes.c_int32),
        _c(lengths, ctypes.c_int32), ctypes.byref(used))
    if rc != 0:
        raise ValueError("page pool or page table too small")
    return K_pool, V_pool, table, lengths, int(used.value)


def compact_write(K_proj, V_proj, keep, cu_seqlens=None, fill=0):
    """Write-side compaction: K_proj,V_proj [T_total,H,D] bf16 bits, keep [H,T_total]
    -> (K_out, V_out [H,T_total,D], lengths[B,H])."""
    K_proj = _u16(K_proj, 3)
    V_proj = _u16(V_proj, 3)
    T_total, H, D = K_proj.shape
    assert V_proj.shape == K_proj.shape
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    assert keep.shape == (H, T_total)
    cu = _cu(cu_seqlens, T_total)
    B = len(cu) - 1
    K_out = np.full((H, T_total, D), fill, dtype=np.uint16)
    V_out = np.full((H, T_total, D), fill, dtype=np.uint16)
    lengths = np.zeros((B, H), dtype=np.int32)
    lib().kvzap_oracle_compact_write(
        _c(K_proj, ctypes.c_uint16), _c(V_proj, ctypes.c_uint16), _c(keep, ctypes.c_uint8),
        _c(cu, ctypes.c_int32), ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(D),
        _c(K_out, ctypes.c_uint16), _c(V_out, ctypes.c_uint16), _c(lengths, ctypes.c_int32))
    return K_out, V_out, lengths


def compact_write_paged(K_proj, V_proj, keep, page_tokens, n_pages_pool, max_pages_per_list,
                        cu_seqlens=None, first_page=0, fill=0):
    """Write-side compaction into pages -> (K_pool, V_pool, page_table, lengths, n_pages_used)."""
    K_proj = _u16(K_proj, 3)
    V_proj = _u16(V_proj, 3)
    T_total, H, D = K_proj.shape
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    assert keep.shape == (H, T_total)
    cu = _cu(cu_seqlens, T_total)
    B = len(cu) - 1
    K_pool = np.full((n_pages_pool, page_tokens, D), fill, dtype=np.uint16)
    V_pool = np.full((n_pages_pool, page_tokens, D), fill, dtype=np.uint16)
    table = np.full((B * H, max_pages_per_list), -1, dtype=np.int32)
    lengths = np.zeros((B, H), dtype=np.int32)
    used = ctypes.c_int32(0)
    rc = lib().kvzap_oracle_compact_write_paged(
        _c(K_proj, ctypes.c_uint16), _c(V_proj, ctypes.c_uint16), _c(keep, ctypes.c_uint8),
        _c(cu, ctypes.c_int32), ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(D),
        ctypes.c_int(page_tokens), ctypes.c_int32(first_page), ctypes.c_int64(n_pages_pool),
        ctypes.c_int(max_pages_per_list),
        _c(K_pool, ctypes.c_uint16), _c(V_pool, ctypes.c_uint16), _c(table, ctypes.c_int32),
        _c(lengths, ctypes.c_int32), ctypes.byref(used))
    if rc != 0:
        raise ValueError("page pool or page table too small")
    return K_pool, V_pool, table, lengths, int(used.value)


def attention(q, K, V, scale):
    """One new token's attention over one pruned list: q [G,D], K,V [n,D] bf16 bits -> out [G,D] fp32."""
    q = _u16(q, 2)
    G, D = q.shape
    K = np.ascontiguousarray(K, dtype=np.uint16).reshape(-1, D)
    V = np.ascontiguousarray(V, dtype=np.uint16).reshape(-1, D)
    assert K.shape == V.shape
    out = np.zeros((G, D), dtype=np.float32)
    rc = lib().kvzap_oracle_attention(_c(q, ctypes.c_uint16), ctypes.c_int(G), _c(K, ctypes.c_uint16),
                                      _c(V, ctypes.c_uint16), ctypes.c_int64(K.shape[0]), ctypes.c_int(D),
                                      ctypes.c_double(scale), _c(out, ctypes.c_float))
    if rc != 0:
        raise MemoryError("oracle attention: out of memory")
    return out


def plan(keep, cu_seqlens=None, page_tokens=0, n_pages_pool=0, max_pages_per_list=1, first_page=0):
    """Write plan: keep [H,T_total] -> (slot [T_total,H] int32, lengths [B,H]) for the dense-ragged layout, or
    (slot, lengths, page_table [B*H,max_pages], n_pages_used) with slot = pool row when page_tokens > 0."""
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    H, T_total = keep.shape
    cu = _cu(cu_seqlens, T_total)
    B = len(cu) - 1
    slot = np.full((T_total, H), -7, dtype=np.int32)
    lengths = np.zeros((B, H), dtype=np.int32)
    table = np.full((B * H, max_pages_per_list), -1, dtype=np.int32)
    used = ctypes.c_int32(0)
    rc = lib().kvzap_oracle_plan(
        _c(keep, ctypes.c_uint8), _c(cu, ctypes.c_int32), ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(page_tokens),
        ctypes.c_int32(first_page), ctypes.c_int64(n_pages_pool), ctypes.c_int(max_pages_per_list),
        _c(slot, ctypes.c_int32), _c(table, ctypes.c_int32), _c(lengths, ctypes.c_int32), ctypes.byref(used))
    if rc != 0:
        raise ValueError("page pool or page table too small")
    if page_tokens > 0:
        return slot, lengths, table, int(used.value)
    return slot, lengths


def e4m3_to_double(bits: int) -> float:
    """Exact value of one E4M3 byte (finite variant; 0x7f and 0xff are NaN)."""
    return float(lib().kvzap_oracle_e4m3_to_double(ctypes.c_uint8(int(bits) & 0xFF)))


def _u8(a, ndim):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint8 and a.ndim == ndim, (a.dtype, a.shape)
    return a


def score_linear_fp8(X8, x_scale, W8, w_scale, b=None):
    """X8 [T,Dh], W8 [H,Dh] E4M3 bytes; x_scale [T], w_scale [H] fp32|None -> scores [T,H] fp32."""
    X8, W8 = _u8(X8, 2), _u8(W8, 2)
    T, Dh = X8.shape
    H = W8.shape[0]
    assert W8.shape[1] == Dh
    x_scale, w_scale, b = _f32_or_none(x_scale, T), _f32_or_none(w_scale, H), _f32_or_none(b, H)
    out = np.empty((T, H), dtype=np.float32)
    lib().kvzap_oracle_score_linear_fp8(
        _c(X8, ctypes.c_uint8), _c(x_scale, ctypes.c_float), ctypes.c_int64(T), ctypes.c_int(Dh),
        _c(W8, ctypes.c_uint8), _c(w_scale, ctypes.c_float), _c(b, ctypes.c_float), ctypes.c_int(H), _c(out, ctypes.c_float))
    return out


def score_mlp_fp8(X8, x_scale, W18, w1_scale, b1, W2, b2):
    """X8 [T,Dh], W18 [N1,Dh] E4M3 bytes with scales [T], [N1]; W2 [H,N1] bf16 bits -> scores [T,H] fp32."""
    X8, W18, W2 = _u8(X8, 2), _u8(W18, 2), _u16(W2, 2)
    T, Dh = X8.shape
    N1, H = W18.shape[0], W2.shape[0]
    assert W18.shape[1] == Dh and W2.shape[1] == N1
    x_scale, w1_scale = _f32_or_none(x_scale, T), _f32_or_none(w1_scale, N1)
    b1, b2 = _f32_or_none(b1, N1), _f32_or_none(b2, H)
    out = np.empty((T, H), dtype=np.float32)
    rc = lib().kvzap_oracle_score_mlp_fp8(
        _c(X8, ctypes.c_uint8), _c(x_scale, ctypes.c_float), ctypes.c_int64(T), ctypes.c_int(Dh),
        _c(W18, ctypes.c_uint8), _c(w1_scale, ctypes.c_float), _c(b1, ctypes.c_float), ctypes.c_int(N1),
        _c(W2, ctypes.c_uint16), _c(b2, ctypes.c_float), ctypes.c_int(H), _c(out, ctypes.c_float))
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return out


def attention_fp8(q, K8, k_scale, V8, v_scale, scale):
    """q [G,D] bf16 bits; K8, V8 [n,D] E4M3 bytes with per-row scales [n] fp32|None -> out [G,D] fp32."""
    q = _u16(q, 2)
    G, D = q.shape
    K8 = np.ascontiguousarray(K8, dtype=np.uint8).reshape(-1, D)
    V8 = np.ascontiguousarray(V8, dtype=np.uint8).reshape(-1, D)
    n = K8.shape[0]
    assert V8.shape == K8.shape
    k_scale, v_scale = _f32_or_none(k_scale, n), _f32_or_none(v_scale, n)
    out = np.zeros((G, D), dtype=np.float32)
    rc = lib().kvzap_oracle_attention_fp8(_c(q, ctypes.c_uint16), ctypes.c_int(G), _c(K8, ctypes.c_uint8),
                                          _c(k_scale, ctypes.c_float), _c(V8, ctypes.c_uint8), _c(v_scale, ctypes.c_float),
                                          ctypes.c_int64(n), ctypes.c_int(D), ctypes.c_double(scale), _c(out, ctypes.c_float))
    if rc != 0:
        raise MemoryError("oracle attention: out of memory")
    return out


def prune_prefill(X, weights, K, V, tau, w, cu_seqlens=None):
    """Algorithm 1 end to end: scores -> window -> threshold -> ordered gather."""
    s = score(X, weights)
    keep = keep_mask(s, tau, w, cu_seqlens)
    K_out, V_out, lengths = compact(K, V, keep, cu_seqlens)
    return s, keep, K_out, V_out, lengths


def layer_flops(H_Q, H, D, Dh, D_int):
    return float(lib().kvzap_oracle_layer_flops(H_Q, H, D, Dh, D_int))


def mlp_flops(Dh, N1, H):
    return float(lib().kvzap_oracle_mlp_flops(Dh, N1, H))


def linear_flops(Dh, H):
    return float(lib().kvzap_oracle_linear_flops(Dh, H))


def param_count(Dh, N1, H):
    return int(lib().kvzap_oracle_param_count(Dh, N1, H))


class DecodeOracle:
    """Decode-time pruning, one list per (sequence, layer, KV head).

    Caption of Algorithm 1 and the contribution list (delayed eviction with a
    sliding window): a token is scored when it is appended; it stays protected
    while it is among the most recent ``w`` tokens; when it leaves that window
    it is dropped iff its buffered score is below tau (kept iff score >= tau),
    and a kept token joins the permanent per-head list, in position order.
    """

    def __init__(self, n_seqs, n_layers, n_heads, head_dim, w):
        assert w >= 0
        self.B, self.L, self.H, self.D, self.w = n_seqs, n_layers, n_heads, head_dim, w
        # permanent part: list of (position, krow, vrow)
        self.prefix = [[[[] for _ in range(n_heads)] for _ in range(n_layers)] for _ in range(n_seqs)]
        # window: deque of (position, score, krow, vrow), oldest first
        self.window = [[[deque() for _ in range(n_heads)] for _ in range(n_layers)] for _ in range(n_seqs)]
        self.n_tokens = np.zeros((n_seqs, n_layers), dtype=np.int64)

    def append(self, b, l, scores_h, k_rows, v_rows, tau):
        """Append one token to sequence b, layer l.  scores_h [H] fp32,
        k_rows/v_rows [H,D] bf16 bits."""
        pos = int(self.n_tokens[b, l])
        tau32 = np.float32(tau)
        for h in range(self.H):
            win = self.window[b][l][h]
            win.append((pos, np.float32(scores_h[h]), np.array(k_rows[h], copy=True),
                        np.array(v_rows[h], copy=True)))
            if len(win) > self.w:
                p, s, kr, vr = win.popleft()
                if s >= tau32:          # NaN compares false -> dropped
                    self.prefix[b][l][h].append((p, kr, vr))
        self.n_tokens[b, l] = pos + 1

    def seed_prefill(self, b, l, scores, K, V, tau):
        """Feed a whole prompt token by token (scores [T,H], K,V [H,T,D])."""
        T = scores.shape[0]
        for t in range(T):
            self.append(b, l, scores[t], K[:, t, :], V[:, t, :], tau)

    def step(self, l, X, weights, K_new, V_new, tau):
        """One decode step for layer l over all sequences.
        X [B,Dh] bf16 bits, K_new,V_new [B,H,D] bf16 bits.  Returns scores [B,H]."""
        s = score(X, weights)
        for b in range(self.B):
            self.append(b, l, s[b], K_new[b], V_new[b], tau)
        return s

    def length(self, b, l, h):
        return len(self.prefix[b][l][h]) + len(self.window[b][l][h])

    def logical(self, b, l, h):
        """(positions [n], K rows [n,D], V rows [n,D]) of the list, position order."""
        items = [(p, kr, vr) for (p, kr, vr) in self.prefix[b][l][h]]
        items += [(p, kr, vr) for (p, _s, kr, vr) in self.window[b][l][h]]
        n = len(items)
        pos = np.array([it[0] for it in items], dtype=np.int64)
        Ko = np.zeros((n, self.D), dtype=np.uint16)
        Vo = np.zeros((n, self.D), dtype=np.uint16)
        for i, it in enumerate(items):
            Ko[i] = it[1]
            Vo[i] = it[2]
        return pos, Ko, Vo

    def window_scores(self, b, l, h):
        return np.array([s for (_p, s, _k, _v) in self.window[b][l][h]], dtype=np.float32)
