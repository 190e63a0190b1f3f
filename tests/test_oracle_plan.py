"""Pins of the oracle's write plan (Discussion, "Implementation Challenges": pruning before the keys and
values are stored): the slot of every kept (token, head) against a running count written out with numpy,
and the property that defines it -- writing every row to its slot reproduces the ordered compaction."""
import numpy as np
import pytest


def _case(seed, seq_lens, H, p_keep=0.4):
    rng = np.random.default_rng(seed)
    T = int(sum(seq_lens))
    keep = (rng.random((H, T)) < p_keep).astype(np.uint8)
    cu = np.zeros(len(seq_lens) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(seq_lens)
    return keep, cu, T


@pytest.mark.parametrize("seq_lens,H", [([13], 3), ([5, 0, 9, 1], 4), ([200, 77], 8)])
def test_plan_dense_is_the_running_count_of_kept_positions(oracle, seq_lens, H):
    keep, cu, T = _case(sum(seq_lens) + H, seq_lens, H)
    slot, lengths = oracle.plan(keep, cu)
    assert slot.shape == (T, H) and slot.dtype == np.int32
    for b in range(len(seq_lens)):
        for h in range(H):
            seg = keep[h, cu[b]:cu[b + 1]].astype(np.int64)
            want = np.where(seg == 1, np.cumsum(seg) - 1, -1)          # exclusive count at kept positions, -1 elsewhere
            np.testing.assert_array_equal(slot[cu[b]:cu[b + 1], h], want)
            assert lengths[b, h] == seg.sum()


@pytest.mark.parametrize("seq_lens,H", [([50], 2), ([31, 64, 0, 7], 8)])
def test_writing_each_row_to_its_slot_gives_the_ordered_compaction(oracle, seq_lens, H):
    keep, cu, T = _case(7, seq_lens, H)
    D = 4
    rng = np.random.default_rng(1)
    K = rng.integers(0, 65535, size=(H, T, D), dtype=np.uint16)
    V = rng.integers(0, 65535, size=(H, T, D), dtype=np.uint16)
    slot, lengths = oracle.plan(keep, cu)
    K_ref, V_ref, len_ref = oracle.compact(K, V, keep, cu, fill=9)
    K_out, V_out = np.full_like(K, 9), np.full_like(V, 9)
    for b in range(len(seq_lens)):
        for t in range(cu[b], cu[b + 1]):
            for h in range(H):
                if slot[t, h] >= 0:
                    K_out[h, cu[b] + slot[t, h]] = K[h, t]
                    V_out[h, cu[b] + slot[t, h]] = V[h, t]
    np.testing.assert_array_equal(lengths, len_ref)
    np.testing.assert_array_equal(K_out, K_ref)
    np.testing.assert_array_equal(V_out, V_ref)


@pytest.mark.parametrize("seq_lens,H,P,first", [([40], 3, 4, 0), ([9, 0, 30, 2], 8, 16, 5), ([64], 2, 7, 1)])
def test_plan_paged_slots_are_the_pool_rows_of_the_paged_compaction(oracle, seq_lens, H, P, first):
    keep, cu, T = _case(3, seq_lens, H, 0.5)
    D = 2
    K = np.arange(H * T * D, dtype=np.uint16).reshape(H, T, D)
    V = K + 7
    n_pool, max_pages = first + H * (T // P + len(seq_lens) + 1), max(seq_lens) // P + 1
    slot, lengths, table, used = oracle.plan(keep, cu, page_tokens=P, n_pages_pool=n_pool, max_pages_per_list=max_pages,
                                             first_page=first)
    Kp, Vp, tab, ln, n_used = oracle.compact_paged(K, V, keep, P, n_pool, max_pages, cu_seqlens=cu, first_page=first, fill=0xFFFF)
    np.testing.assert_array_equal(lengths, ln)
    np.testing.assert_array_equal(table, tab)
    assert used == n_used
    pool_k = np.full((n_pool * P, D), 0xFFFF, dtype=np.uint16)
    pool_v = np.full((n_pool * P, D), 0xFFFF, dtype=np.uint16)
    rows = set()
    for t in range(T):
        for h in range(H):
            if keep[h, t]:
                r = int(slot[t, h])
                assert first * P <= r < (first + used) * P and r not in rows     # inside the assigned pages, no row twice
                rows.add(r)
                pool_k[r], pool_v[r] = K[h, t], V[h, t]
            else:
                assert slot[t, h] == -1
    np.testing.assert_array_equal(pool_k.reshape(n_pool, P, D), Kp)
    np.testing.assert_array_equal(pool_v.reshape(n_pool, P, D), Vp)


def test_plan_paged_pool_too_small_is_an_error(oracle):
    keep = np.ones((2, 40), dtype=np.uint8)
    with pytest.raises(ValueError):
        oracle.plan(keep, None, page_tokens=4, n_pages_pool=19, max_pages_per_list=10)
    with pytest.raises(ValueError):
        oracle.plan(keep, None, page_tokens=4, n_pages_pool=100, max_pages_per_list=9)


def test_plan_all_kept_and_none_kept(oracle):
    T, H = 11, 2
    slot, lengths = oracle.plan(np.ones((H, T), dtype=np.uint8))
    np.testing.assert_array_equal(slot, np.tile(np.arange(T, dtype=np.int32)[:, None], (1, H)))
    assert (lengths == T).all()
    slot, lengths = oracle.plan(np.zeros((H, T), dtype=np.uint8))
    assert (slot == -1).all() and (lengths == 0).all()
