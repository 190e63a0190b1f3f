"""Pins for the oracle's fixed-budget (top-k) selection (CPU only): numpy sorts and counts."""
import numpy as np
import pytest


def _scores(rng, T, H):
    return rng.standard_normal((T, H)).astype(np.float32)


@pytest.mark.parametrize("per_layer", [False, True])
@pytest.mark.parametrize("lens,w,ratio", [([300], 16, 0.25), ([50, 1, 0, 130, 17], 16, 0.4), ([64], 0, 0.1), ([40], 64, 0.5)])
def test_topk_mask_is_the_k_largest_by_numpy_sort(oracle, lens, w, ratio, per_layer):
    rng = np.random.default_rng(sum(lens) + w)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T, H = int(cu[-1]), 5
    s = _scores(rng, T, H)
    keep, tau = oracle.topk_mask(s, ratio, w, per_layer, cu)
    r = float(np.float32(ratio))
    for b, Tb in enumerate(lens):
        t0 = int(cu[b])
        n_cand = max(Tb - w, 0)
        k = int(np.ceil(r * n_cand))
        cand = s[t0:t0 + n_cand]                                   # [n_cand, H]
        assert keep[:, t0 + n_cand:t0 + Tb].all()                  # the window is kept whatever the scores
        if per_layer:
            chosen = np.zeros_like(cand, dtype=bool)
            if k > 0:
                order = np.argsort(-cand, axis=None, kind="stable")[:k * H]
                chosen.flat[order] = True
            np.testing.assert_array_equal(keep[:, t0:t0 + n_cand].T.astype(bool), chosen)
            assert chosen.sum() == k * H                           # no ties in random normals: the budget exactly
            assert (tau[b] == tau[b, 0]).all()
        else:
            for h in range(H):
                chosen = np.zeros(n_cand, dtype=bool)
                if k > 0:
                    chosen[np.argsort(-cand[:, h], kind="stable")[:k]] = True
                np.testing.assert_array_equal(keep[h, t0:t0 + n_cand].astype(bool), chosen)
                assert chosen.sum() == k
                if k > 0:
                    assert tau[b, h] == np.sort(cand[:, h])[::-1][k - 1]
                else:
                    assert tau[b, h] == np.inf


def test_topk_ties_nan_and_extremes(oracle):
    T, H, w = 40, 2, 4
    s = np.zeros((T, H), dtype=np.float32)
    s[:, 0] = np.arange(T) % 4                    # values 0..3, nine of each among the 36 candidates
    s[:, 1] = np.linspace(-1, 1, T)
    s[5, 1] = np.nan
    s[6, 1] = np.inf
    keep, tau = oracle.topk_mask(s, 0.25, w)      # k = 9
    assert tau[0, 0] == 3.0 and keep[0, :36].sum() == 9            # exactly the nine 3s
    keep, tau = oracle.topk_mask(s, 10 / 36, w)   # k = 10: the cut value 2 brings all nine 2s along
    assert tau[0, 0] == 2.0 and keep[0, :36].sum() == 18
    assert keep[1, 6] == 1 and keep[1, 5] == 0                     # +inf first, NaN never
    keep, tau = oracle.topk_mask(s, 0.0, w)       # no budget: the window alone
    assert np.isposinf(tau).all() and keep[0].sum() == w and keep[1].sum() == w + 1   # (+inf >= +inf is kept)
    keep, tau = oracle.topk_mask(s, 1.0, w)       # everything that is a number
    assert tau[0, 0] == 0.0 and keep[0].all()
    assert np.isneginf(tau[0, 1]) and keep[1].sum() == T - 1 and keep[1, 5] == 0   # 35 numbers for a budget of 36
    # a larger budget keeps a superset; per-layer with one head is per-head
    a, _ = oracle.topk_mask(s, 0.2, w)
    b, _ = oracle.topk_mask(s, 0.6, w)
    assert ((a == 1) <= (b == 1)).all()
    one = s[:, :1].copy()
    np.testing.assert_array_equal(oracle.topk_mask(one, 0.3, w, False)[0], oracle.topk_mask(one, 0.3, w, True)[0])


def test_topk_equals_threshold_mask_at_its_cut_value(oracle):
    rng = np.random.default_rng(8)
    s = _scores(rng, 200, 3)
    keep, tau = oracle.topk_mask(s, 0.3, 16)
    for h in range(3):
        one_head = oracle.keep_mask(s[:, h:h + 1], float(tau[0, h]), 16)
        np.testing.assert_array_equal(keep[h], one_head[0])
