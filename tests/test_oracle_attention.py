"""Pins for the oracle's attention over a pruned list (CPU only).

The operation is ordinary scaled dot-product softmax attention of one new token over a
list of any length; each test checks it against something other than itself: a library
composition in fp64, closed forms and invariants.
"""
import numpy as np
import pytest
import torch


def _bf16_bits(x):
    """float array -> bf16 bit patterns (round to nearest even, via torch) and the rounded values."""
    t = torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy(), t.to(torch.float64).numpy()


@pytest.mark.parametrize("G,n,D", [(4, 37, 16), (1, 1, 8), (8, 300, 128), (3, 129, 64)])
def test_attention_matches_torch_fp64_softmax_composition(oracle, G, n, D):
    rng = np.random.default_rng(G * 1000 + n)
    qb, q = _bf16_bits(rng.standard_normal((G, D)))
    Kb, K = _bf16_bits(rng.standard_normal((n, D)))
    Vb, V = _bf16_bits(rng.standard_normal((n, D)))
    scale = 1.0 / np.sqrt(D)
    want = torch.softmax(torch.from_numpy(q) @ torch.from_numpy(K).T * scale, dim=-1) @ torch.from_numpy(V)
    got = oracle.attention(qb, Kb, Vb, scale)
    np.testing.assert_allclose(got, want.numpy(), rtol=0, atol=2e-7)      # one fp32 rounding of an O(1) value


def test_attention_closed_forms(oracle):
    rng = np.random.default_rng(5)
    G, n, D = 2, 50, 16
    qb, q = _bf16_bits(rng.standard_normal((G, D)))
    Vb, V = _bf16_bits(rng.standard_normal((n, D)))
    # identical keys: every weight is 1/n, the output is the mean of the value rows
    Kb, _ = _bf16_bits(np.tile(rng.standard_normal((1, D)), (n, 1)))
    np.testing.assert_allclose(oracle.attention(qb, Kb, Vb, 0.25), np.tile(V.mean(0), (G, 1)), atol=1e-6)
    # scale 0: again uniform weights, whatever the keys
    Kb2, _ = _bf16_bits(rng.standard_normal((n, D)))
    np.testing.assert_allclose(oracle.attention(qb, Kb2, Vb, 0.0), np.tile(V.mean(0), (G, 1)), atol=1e-6)
    # a single row: the output is that value row exactly, for every query
    np.testing.assert_array_equal(oracle.attention(qb, Kb2[:1], Vb[:1], 3.0), np.tile(V[:1].astype(np.float32), (G, 1)))
    # an empty list gives zeros
    assert (oracle.attention(qb, Kb2[:0], Vb[:0], 1.0) == 0).all()
    # one key that dominates (q = e_0 * 8, that key = e_0 * 64, others ~ 0): its value row comes out
    q1 = np.zeros((1, D)); q1[0, 0] = 8.0
    K1 = np.zeros((n, D)); K1[17, 0] = 64.0
    out = oracle.attention(_bf16_bits(q1)[0], _bf16_bits(K1)[0], Vb, 1.0)
    np.testing.assert_allclose(out[0], V[17], atol=1e-6)
    # two keys with equal logits, all others far below: the mean of their two value rows
    K2 = np.full((n, D), 0.0); K2[3, 0] = 4.0; K2[40, 0] = 4.0
    K2[np.setdiff1d(np.arange(n), [3, 40]), 0] = -64.0
    out = oracle.attention(_bf16_bits(q1)[0], _bf16_bits(K2)[0], Vb, 1.0)
    np.testing.assert_allclose(out[0], 0.5 * (V[3] + V[40]), atol=1e-6)


def test_attention_invariants(oracle):
    rng = np.random.default_rng(6)
    G, n, D = 4, 90, 32
    qb, q = _bf16_bits(rng.standard_normal((G, D)))
    Kb, K = _bf16_bits(rng.standard_normal((n, D)))
    Vb, V = _bf16_bits(rng.standard_normal((n, D)))
    base = oracle.attention(qb, Kb, Vb, 0.3)
    # the order of the list's rows does not matter (the pruned cache keeps prefix and window apart)
    perm = rng.permutation(n)
    np.testing.assert_allclose(oracle.attention(qb, Kb[perm], Vb[perm], 0.3), base, atol=1e-6)
    # queries are independent: one query alone gives its row of the joint result
    for g in range(G):
        np.testing.assert_array_equal(oracle.attention(qb[g:g + 1], Kb, Vb, 0.3), base[g:g + 1])
    # the output is a convex combination of the value rows
    assert (base <= V.max(0) + 1e-6).all() and (base >= V.min(0) - 1e-6).all()
    # K and V are not interchangeable, and the scale matters
    assert np.abs(oracle.attention(qb, Vb, Kb, 0.3) - base).max() > 1e-2
    assert np.abs(oracle.attention(qb, Kb, Vb, 0.6) - base).max() > 1e-3
    # duplicating the whole list changes nothing (weights halve, rows double)
    np.testing.assert_allclose(oracle.attention(qb, np.concatenate([Kb, Kb]), np.concatenate([Vb, Vb]), 0.3), base,
                               atol=1e-6)
    # a row removed from the list (pruned) changes the output by at most its weight times the value range
    p = torch.softmax(torch.from_numpy(q) @ torch.from_numpy(K).T * 0.3, dim=-1).numpy()
    drop = int(np.argmin(p.max(0)))
    keep = np.setdiff1d(np.arange(n), [drop])
    pruned = oracle.attention(qb, Kb[keep], Vb[keep], 0.3)
    bound = p[:, drop:drop + 1] * (V.max(0) - V.min(0))[None, :] / (1 - p[:, drop:drop + 1])
    assert (np.abs(pruned - base) <= bound + 1e-6).all()
