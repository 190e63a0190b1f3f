"""Pins for the oracle's window/threshold mask, compaction and decode rule (CPU only).

Each test states a property the paper fixes (Method, "KVzap"; Algorithm 1 and
its caption) or a brute-force restatement on small inputs.
"""
import numpy as np
import pytest


def _scores(rng, T, H):
    return rng.standard_normal((T, H)).astype(np.float32)


def _tagged_kv(H, T, D):
    """Rows whose contents encode (head, position) so order and source are checkable."""
    K = np.zeros((H, T, D), dtype=np.uint16)
    V = np.zeros((H, T, D), dtype=np.uint16)
    for h in range(H):
        K[h, :, 0] = h
        V[h, :, 0] = h + 100
        K[h, :, 1] = np.arange(T) & 0xFFFF
        V[h, :, 1] = np.arange(T) & 0xFFFF
        K[h, :, 2:] = (np.arange(T)[:, None] * 7 + np.arange(D - 2)[None, :] + h) & 0xFFFF
        V[h, :, 2:] = (np.arange(T)[:, None] * 13 + np.arange(D - 2)[None, :] + 3 * h) & 0xFFFF
    return K, V


def test_mask_is_window_or_threshold_brute_force(oracle):
    rng = np.random.default_rng(0)
    T, H, w, tau = 300, 8, 128, 0.43
    s = _scores(rng, T, H)
    keep = oracle.keep_mask(s, tau, w)
    assert keep.shape == (H, T) and keep.dtype == np.uint8
    for h in range(H):
        for t in range(T):
            want = (t >= T - w) or (s[t, h] >= np.float32(tau))
            assert keep[h, t] == want
    # last w positions kept for every head, whatever the scores
    assert keep[:, T - w:].all()
    # heads are independent: permuting the score columns permutes the mask rows
    perm = rng.permutation(H)
    np.testing.assert_array_equal(oracle.keep_mask(s[:, perm], tau, w), keep[perm])


def test_mask_tie_is_kept_and_nan_is_dropped(oracle):
    s = np.array([[0.43, np.nan, np.inf, -np.inf]] * 3, dtype=np.float32)
    keep = oracle.keep_mask(s, np.float32(0.43), 0)
    np.testing.assert_array_equal(keep[:, 0], [1, 0, 1, 0])
    # NaN inside the window is still kept
    keep = oracle.keep_mask(s, 0.43, 1)
    np.testing.assert_array_equal(keep[:, 2], [1, 1, 1, 1])
    np.testing.assert_array_equal(keep[:, 1], [1, 0, 1, 0])


@pytest.mark.parametrize("T,w", [(1, 128), (127, 128), (128, 128), (129, 128), (50, 0), (50, 512), (0, 4)])
def test_mask_window_edge_cases(oracle, T, w):
    rng = np.random.default_rng(T + w)
    H = 3
    s = _scores(rng, T, H)
    # tau = +inf keeps exactly the window, tau = -inf keeps everything (no NaNs here)
    only_window = oracle.keep_mask(s, np.inf, w)
    assert only_window.sum() == H * min(w, T)
    if T:
        assert only_window[:, max(T - w, 0):].all() and not only_window[:, :max(T - w, 0)].any()
    assert oracle.keep_mask(s, -np.inf, w).sum() == H * T
    if w == 0 and T:
        np.testing.assert_array_equal(oracle.keep_mask(s, 0.0, 0), (s.T >= 0).astype(np.uint8))


def test_larger_tau_keeps_a_subset(oracle):
    rng = np.random.default_rng(7)
    s = _scores(rng, 1000, 8)
    prev = None
    for tau in [-2.0, 0.0, 0.43, 0.84, 3.0]:
        keep = oracle.keep_mask(s, tau, 64).astype(bool)
        if prev is not None:
            assert not (keep & ~prev).any()          # kept(tau2) subset of kept(tau1), tau2 > tau1
            assert keep.sum() < prev.sum()
        prev = keep


def test_keep_fraction_of_unit_normal_scores(oracle):
    # recipe check: tau = 0.43 keeps about one third of N(0,1) scores
    s = _scores(np.random.default_rng(8), 20000, 8)
    frac = oracle.keep_mask(s, 0.43, 0).mean()
    assert abs(frac - 0.3336) < 0.01


def test_window_is_per_sequence(oracle):
    rng = np.random.default_rng(9)
    lens = [5, 40, 1, 0, 17]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T, H, w = int(cu[-1]), 2, 8
    s = _scores(rng, T, H)
    keep = oracle.keep_mask(s, 10.0, w, cu)              # nothing passes the threshold
    for b, n in enumerate(lens):
        seg = keep[:, cu[b]:cu[b + 1]]
        assert seg.sum() == H * min(n, w)
        if n:
            assert seg[:, max(n - w, 0):].all()
    # each sequence alone gives the same mask as inside the packed batch
    full = oracle.keep_mask(s, 0.2, w, cu)
    for b in range(len(lens)):
        alone = oracle.keep_mask(s[cu[b]:cu[b + 1]], 0.2, w)
        np.testing.assert_array_equal(full[:, cu[b]:cu[b + 1]], alone)


def test_compaction_is_the_ordered_gather(oracle):
    rng = np.random.default_rng(10)
    H, T, D = 4, 333, 16
    K, V = _tagged_kv(H, T, D)
    keep = (rng.random((H, T)) < 0.35).astype(np.uint8)
    POISON = 0xDEAD
    K_out, V_out, lengths = oracle.compact(K, V, keep, fill=POISON)
    assert lengths.shape == (1, H)
    for h in range(H):
        idx = np.flatnonzero(keep[h])                     # explicit index list, increasing
        n = len(idx)
        assert lengths[0, h] == n == int(keep[h].sum())   # kept count == mask popcount
        np.testing.assert_array_equal(K_out[h, :n], K[h, idx])     # keys[indices]
        np.testing.assert_array_equal(V_out[h, :n], V[h, idx])     # values[indices], same indices
        assert np.all(np.diff(K_out[h, :n, 1].astype(np.int64)) > 0)   # token order preserved
        assert (K_out[h, n:] == POISON).all() and (V_out[h, n:] == POISON).all()   # untouched tail
        assert (K_out[h, :n, 0] == h).all() and (V_out[h, :n, 0] == h + 100).all()  # no head mixing


def test_compaction_all_kept_is_identity_and_none_kept_is_empty(oracle):
    K, V = _tagged_kv(3, 65, 8)
    K_out, V_out, lengths = oracle.compact(K, V, np.ones((3, 65), np.uint8))
    np.testing.assert_array_equal(K_out, K)
    np.testing.assert_array_equal(V_out, V)
    assert (lengths == 65).all()
    K_out, V_out, lengths = oracle.compact(K, V, np.zeros((3, 65), np.uint8), fill=0xBEEF)
    assert (lengths == 0).all() and (K_out == 0xBEEF).all() and (V_out == 0xBEEF).all()


def test_compaction_multi_sequence_lists_start_at_sequence_start(oracle):
    rng = np.random.default_rng(11)
    lens = [30, 1, 0, 100, 9]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    H, T, D = 2, int(cu[-1]), 8
    K, V = _tagged_kv(H, T, D)
    keep = (rng.random((H, T)) < 0.5).astype(np.uint8)
    K_out, V_out, lengths = oracle.compact(K, V, keep, cu, fill=0xAAAA)
    assert lengths.shape == (len(lens), H)
    for b in range(len(lens)):
        for h in range(H):
            idx = cu[b] + np.flatnonzero(keep[h, cu[b]:cu[b + 1]])
            n = len(idx)
            assert lengths[b, h] == n
            np.testing.assert_array_equal(K_out[h, cu[b]:cu[b] + n], K[h, idx])
            np.testing.assert_array_equal(V_out[h, cu[b]:cu[b] + n], V[h, idx])
            assert (K_out[h, cu[b] + n:cu[b + 1]] == 0xAAAA).all()


def test_paged_compaction_matches_dense_and_assigns_pages_in_list_order(oracle):
    rng = np.random.default_rng(12)
    lens = [37, 64, 5]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    H, T, D, P = 3, int(cu[-1]), 8, 16
    K, V = _tagged_kv(H, T, D)
    keep = (rng.random((H, T)) < 0.6).astype(np.uint8)
    Kd, Vd, len_d = oracle.compact(K, V, keep, cu)
    Kp, Vp, table, len_p, used = oracle.compact_paged(K, V, keep, P, n_pages_pool=40, max_pages_per_list=5,
                                                      cu_seqlens=cu, first_page=2, fill=0x1111)
    np.testing.assert_array_equal(len_p, len_d)
    cursor = 2
    for b in range(len(lens)):
        for h in range(H):
            n = int(len_d[b, h])
            need = -(-n // P)
            pages = table[b * H + h]
            np.testing.assert_array_equal(pages[:need], np.arange(cursor, cursor + need))
            assert (pages[need:] == -1).all()
            cursor += need
            rows_k = Kp[pages[:need]].reshape(-1, D)[:n]
            rows_v = Vp[pages[:need]].reshape(-1, D)[:n]
            np.testing.assert_array_equal(rows_k, Kd[h, cu[b]:cu[b] + n])
            np.testing.assert_array_equal(rows_v, Vd[h, cu[b]:cu[b] + n])
    assert used == cursor - 2
    assert (Kp[:2] == 0x1111).all() and (Kp[cursor:] == 0x1111).all()
    with pytest.raises(ValueError):
        oracle.compact_paged(K, V, keep, P, n_pages_pool=used + 1, max_pages_per_list=5, cu_seqlens=cu, first_page=2)
    with pytest.raises(ValueError):
        oracle.compact_paged(K, V, keep, P, n_pages_pool=40, max_pages_per_list=1, cu_seqlens=cu)


@pytest.mark.parametrize("w", [0, 1, 5, 16])
def test_decode_equals_prefill_on_the_concatenation(oracle, w):
    rng = np.random.default_rng(20 + w)
    H, D, tau = 3, 8, 0.1
    T_total = 60
    s = _scores(rng, T_total, H)
    s[7, 1] = np.nan
    s[9, 0] = np.float32(tau)                     # tie -> kept
    K, V = _tagged_kv(H, T_total, D)
    dec = oracle.DecodeOracle(1, 1, H, D, w)
    prev_len = [0] * H
    for n in range(1, T_total + 1):
        dec.append(0, 0, s[n - 1], K[:, n - 1], V[:, n - 1], tau)
        keep = oracle.keep_mask(s[:n], tau, w)
        Kc, Vc, lengths = oracle.compact(K[:, :n], V[:, :n], keep)
        for h in range(H):
            pos, Kd, Vd = dec.logical(0, 0, h)
            L = int(lengths[0, h])
            assert dec.length(0, 0, h) == L
            np.testing.assert_array_equal(pos, np.flatnonzero(keep[h]))
            np.testing.assert_array_equal(Kd, Kc[h, :L])
            np.testing.assert_array_equal(Vd, Vc[h, :L])
            # one token in; at most the one leaving the window goes out
            exited = n - w - 1
            dropped = exited >= 0 and not (s[exited, h] >= np.float32(tau))
            assert L == prev_len[h] + 1 - int(dropped)
            prev_len[h] = L
            # the score buffer holds exactly the window's scores
            np.testing.assert_array_equal(dec.window_scores(0, 0, h), s[max(n - w, 0):n, h])


def test_decode_prefill_then_steps_equals_longer_prefill(oracle):
    rng = np.random.default_rng(30)
    H, D, w, tau, T0, k = 2, 8, 4, -0.2, 21, 9
    s = _scores(rng, T0 + k, H)
    K, V = _tagged_kv(H, T0 + k, D)
    dec = oracle.DecodeOracle(1, 1, H, D, w)
    dec.seed_prefill(0, 0, s[:T0], K[:, :T0], V[:, :T0], tau)
    for t in range(T0, T0 + k):
        dec.append(0, 0, s[t], K[:, t], V[:, t], tau)
    keep = oracle.keep_mask(s, tau, w)
    Kc, Vc, lengths = oracle.compact(K, V, keep)
    for h in range(H):
        _pos, Kd, Vd = dec.logical(0, 0, h)
        np.testing.assert_array_equal(Kd, Kc[h, :lengths[0, h]])
        np.testing.assert_array_equal(Vd, Vc[h, :lengths[0, h]])


# ---------------------------------------------------------------------------
# Write-side pruning (Discussion, "Implementation Challenges"): K and V arrive as
# the projection wrote them, [T, H, D].


def test_write_side_compaction_is_the_ordered_gather_of_projection_rows(oracle):
    rng = np.random.default_rng(40)
    lens = [50, 0, 3, 120]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    H, T, D = 3, int(cu[-1]), 8
    K, V = _tagged_kv(H, T, D)
    K_proj = np.ascontiguousarray(K.transpose(1, 0, 2))      # [T, H, D]
    V_proj = np.ascontiguousarray(V.transpose(1, 0, 2))
    keep = (rng.random((H, T)) < 0.4).astype(np.uint8)
    K_out, V_out, lengths = oracle.compact_write(K_proj, V_proj, keep, cu, fill=0xDEAD)
    for b in range(len(lens)):
        for h in range(H):
            idx = cu[b] + np.flatnonzero(keep[h, cu[b]:cu[b + 1]])       # explicit index list
            n = len(idx)
            assert lengths[b, h] == n
            np.testing.assert_array_equal(K_out[h, cu[b]:cu[b] + n], K_proj[idx, h])
            np.testing.assert_array_equal(V_out[h, cu[b]:cu[b] + n], V_proj[idx, h])
            assert (K_out[h, cu[b]:cu[b] + n, 0] == h).all()             # rows of head h only
            assert np.all(np.diff(K_out[h, cu[b]:cu[b] + n, 1].astype(np.int64)) > 0)   # token order
            assert (K_out[h, cu[b] + n:cu[b + 1]] == 0xDEAD).all()
            assert (V_out[h, cu[b] + n:cu[b + 1]] == 0xDEAD).all()
    # keeping everything is the transposition [T,H,D] -> [H,T,D]
    K_all, V_all, len_all = oracle.compact_write(K_proj, V_proj, np.ones((H, T), np.uint8), cu)
    np.testing.assert_array_equal(K_all, K)
    np.testing.assert_array_equal(V_all, V)
    np.testing.assert_array_equal(len_all, np.repeat(np.array(lens)[:, None], H, 1))


def test_write_side_paged_compaction_pages_and_rows(oracle):
    rng = np.random.default_rng(41)
    lens = [37, 64, 5]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    H, T, D, P = 3, int(cu[-1]), 8, 16
    K, V = _tagged_kv(H, T, D)
    K_proj = np.ascontiguousarray(K.transpose(1, 0, 2))
    V_proj = np.ascontiguousarray(V.transpose(1, 0, 2))
    keep = (rng.random((H, T)) < 0.6).astype(np.uint8)
    Kp, Vp, table, lengths, used = oracle.compact_write_paged(K_proj, V_proj, keep, P, n_pages_pool=40,
                                                              max_pages_per_list=5, cu_seqlens=cu, first_page=2,
                                                              fill=0x1111)
    cursor = 2
    for b in range(len(lens)):
        for h in range(H):
            idx = cu[b] + np.flatnonzero(keep[h, cu[b]:cu[b + 1]])
            n, need = len(idx), -(-len(idx) // P)
            assert lengths[b, h] == n
            pages = table[b * H + h]
            np.testing.assert_array_equal(pages[:need], np.arange(cursor, cursor + need))   # (b,h) order, contiguous
            assert (pages[need:] == -1).all()
            np.testing.assert_array_equal(Kp[pages[:need]].reshape(-1, D)[:n], K_proj[idx, h])
            np.testing.assert_array_equal(Vp[pages[:need]].reshape(-1, D)[:n], V_proj[idx, h])
            cursor += need
    assert used == cursor - 2
    assert (Kp[:2] == 0x1111).all() and (Kp[cursor:] == 0x1111).all()
    with pytest.raises(ValueError):
        oracle.compact_write_paged(K_proj, V_proj, keep, P, n_pages_pool=used + 1, max_pages_per_list=5,
                                   cu_seqlens=cu, first_page=2)
    with pytest.raises(ValueError):
        oracle.compact_write_paged(K_proj, V_proj, keep, P, n_pages_pool=40, max_pages_per_list=1, cu_seqlens=cu)
