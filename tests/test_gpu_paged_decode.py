"""GPU parity for the paged prefill output and the decode step, against the CPU oracle.

Paged prefill: deterministic page assignment, so pools, page tables and lengths are
compared bit for bit with the oracle run on the GPU's own scores.
Decode: scores are compared within the tolerance; the eviction decisions and the list
contents are compared bit for bit with the decode oracle fed the GPU's own scores (any
unique in-range page is a valid allocation, so lists are compared through the export call
and the page tables are checked for validity, not for equality).
"""
import numpy as np
import pytest
import torch

from paper_2601_07891_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2601_07891_b200 import binding as b
    b.load()
    return b


def _weights(d_model, hidden, H, seed, bias_sigma=0.3):
    if hidden == 0:
        return synth.linear_weights(d_model, H, seed, "cpu", bias_sigma)
    return synth.mlp_weights(d_model, hidden, H, seed, "cpu", bias_sigma)


@pytest.mark.parametrize("seq_lens,hidden,P", [([700], 0, 16), ([37, 64, 5, 0, 300], 128, 16), ([1000, 24], 0, 7)])
def test_paged_prefill_matches_oracle(binding, oracle, seq_lens, hidden, P):
    d_model, H, D, tau, w = 256, 8, 64, 0.3, 16
    T, B = int(sum(seq_lens)), len(seq_lens)
    ctx = binding.Kvzap(d_model, hidden, H, D, 1, T, max_seqs=B)
    weights = _weights(d_model, hidden, H, seed=B + hidden)
    ctx.set_weights(0, *[parity.dev(x) for x in weights])
    X = synth.hidden_states(T, d_model, seed=5)
    K, V = synth.keys_values(H, T, D, seed=6)
    cu = synth.cu_seqlens(seq_lens)
    cu_dev = torch.from_numpy(cu).cuda() if B > 1 else None
    n_pool, max_pages, first_page = H * (T // P + B + 1) + 5, max(seq_lens) // P + 2, 3
    pool = lambda: torch.full((n_pool, P, D), -5.0, dtype=torch.bfloat16, device="cuda")
    K_pool, V_pool = pool(), pool()
    table = torch.full((B * H, max_pages), -1, dtype=torch.int32, device="cuda")
    lengths = torch.zeros(B, H, dtype=torch.int32, device="cuda")
    used = torch.zeros(1, dtype=torch.int32, device="cuda")
    scores = torch.empty(T, H, dtype=torch.float32, device="cuda")
    binding.kvzap_prefill_fused_paged(ctx.handle, 0, parity.dev(X), parity.dev(K), parity.dev(V), cu_dev, B, tau, w,
                                      K_pool, V_pool, P, first_page, table, lengths, used, scores)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    want, _ = parity.check_scores(oracle, scores, X, weights)
    s = scores.cpu().numpy()
    cu_arg = cu if B > 1 else None
    keep = parity.check_mask_band(oracle, s, want, tau, w, cu_arg)
    fill = int(synth.bits(torch.tensor([-5.0], dtype=torch.bfloat16))[0])
    Kp, Vp, tab, ln, n_used = oracle.compact_paged(synth.bits(K), synth.bits(V), keep, P, n_pool, max_pages,
                                                   cu_seqlens=cu_arg, first_page=first_page, fill=fill)
    np.testing.assert_array_equal(lengths.cpu().numpy(), ln)
    assert int(used.item()) == n_used
    np.testing.assert_array_equal(table.cpu().numpy(), tab)
    np.testing.assert_array_equal(synth.bits(K_pool), Kp)       # untouched pages keep their fill
    np.testing.assert_array_equal(synth.bits(V_pool), Vp)
    # two-call route gives the same bits
    K2, V2 = pool(), pool()
    table2 = torch.full_like(table, -1)
    len2, used2 = torch.zeros_like(lengths), torch.zeros_like(used)
    binding.kvzap_prune_prefill_paged(ctx.handle, parity.dev(K), parity.dev(V), scores, cu_dev, B, tau, w, K2, V2, P,
                                      first_page, table2, len2, used2)
    torch.cuda.synchronize()
    assert torch.equal(table2, table) and torch.equal(len2, lengths) and torch.equal(used2, used)
    assert torch.equal(K2.view(torch.int16), K_pool.view(torch.int16))
    assert torch.equal(V2.view(torch.int16), V_pool.view(torch.int16))
    ctx.close()


def test_paged_prefill_pool_too_small_sets_status_and_writes_nothing(binding, oracle):
    H, D, T, P = 8, 64, 500, 16
    ctx = binding.Kvzap(256, 0, H, D, 1, T)
    K, V = synth.keys_values(H, T, D, seed=1)
    scores = torch.randn(T, H, generator=torch.Generator().manual_seed(2)).cuda()
    pool = torch.full((10, P, D), -5.0, dtype=torch.bfloat16, device="cuda")      # far too few pages
    V_pool = pool.clone()
    table = torch.full((H, 40), -1, dtype=torch.int32, device="cuda")
    lengths = torch.zeros(1, H, dtype=torch.int32, device="cuda")
    used = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    binding.kvzap_prune_prefill_paged(ctx.handle, parity.dev(K), parity.dev(V), scores, None, 1, 0.0, 8, pool, V_pool, P,
                                      0, table, lengths, used)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 4                       # KVZAP_ERR_OOM_PAGES, and the word is cleared by the poll
    assert ctx.poll_status() == 0
    assert int(used.item()) == 0 and (pool == -5.0).all() and (V_pool == -5.0).all()
    keep = oracle.keep_mask(scores.cpu().numpy(), 0.0, 8)
    np.testing.assert_array_equal(lengths.cpu().numpy()[0], keep.sum(axis=1))
    ctx.close()


def _export(binding, ctx, cache, b, l, h, cap, D):
    K_out = torch.zeros(cap, D, dtype=torch.bfloat16, device="cuda")
    V_out = torch.zeros(cap, D, dtype=torch.bfloat16, device="cuda")
    n = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.kvzap_cache_export(ctx.handle, cache, b, l, h, K_out, V_out, n)
    torch.cuda.synchronize()
    n = int(n.item())
    return synth.bits(K_out)[:n], synth.bits(V_out)[:n], n


def _check_cache_against_oracle(binding, oracle, ctx, cache, dec, B, L, H, D, cap, P, n_pool):
    lengths = torch.zeros(B, L, H, dtype=torch.int32, device="cuda")
    binding.kvzap_cache_lengths(ctx.handle, cache, lengths)
    torch.cuda.synchronize()
    ln = lengths.cpu().numpy()
    for b in range(B):
        for l in range(L):
            for h in range(H):
                _pos, Kd, Vd = dec.logical(b, l, h)
                assert ln[b, l, h] == dec.length(b, l, h) == len(Kd)
                Kg, Vg, n = _export(binding, ctx, cache, b, l, h, cap, D)
                assert n == len(Kd)
                np.testing.assert_array_equal(Kg, Kd)
                np.testing.assert_array_equal(Vg, Vd)


@pytest.mark.parametrize("hidden,w,P,B,L", [(128, 8, 4, 3, 2), (0, 5, 16, 2, 1), (512, 0, 4, 2, 2), (64, 16, 3, 130, 1)])
def test_decode_steps_match_decode_oracle(binding, oracle, hidden, w, P, B, L):
    d_model, H, D, tau, n_steps = 256, 8, 64, 0.1, 40 if B < 100 else 20
    ctx = binding.Kvzap(d_model, hidden, H, D, L, max_tokens=max(B, 128), max_seqs=1)
    all_w = []
    for l in range(L):
        wts = _weights(d_model, hidden, H, seed=50 + l)
        all_w.append(wts)
        ctx.set_weights(l, *[parity.dev(x) for x in wts])
    n_pool = B * L * H * (n_steps // P + 2)
    K_pool = torch.zeros(n_pool, P, D, dtype=torch.bfloat16, device="cuda")
    V_pool = torch.zeros(n_pool, P, D, dtype=torch.bfloat16, device="cuda")
    max_pages = n_steps // P + 2
    cache = binding.kvzap_cache_create(ctx.handle, B, w, P, K_pool, V_pool, max_pages)
    dec = oracle.DecodeOracle(B, L, H, D, w)
    worst = 0.0
    for step in range(n_steps):
        X = synth.hidden_states(L * B, d_model, seed=1000 + step).view(L, B, d_model)
        K_new, V_new = synth.keys_values(L * B, H, D, seed=2000 + step)       # [L*B, H, D]
        K_new, V_new = K_new.view(L, B, H, D), V_new.view(L, B, H, D)
        scores = torch.empty(L, B, H, dtype=torch.float32, device="cuda")
        binding.kvzap_decode_step(ctx.handle, cache, 0, L, parity.dev(X), parity.dev(K_new), parity.dev(V_new), tau,
                                  scores if step % 2 == 0 else None)
        if step % 2 == 1:      # scores not requested: recompute them through the scoring call for the oracle
            for l in range(L):
                ctx.score(l, parity.dev(X[l]), out=scores[l])
        torch.cuda.synchronize()
        s = scores.cpu().numpy()
        for l in range(L):
            want = oracle.score(synth.bits(X[l]), parity.weights_to_oracle(all_w[l]))
            worst = max(worst, float(np.abs(s[l] - want).max()))
            Kb, Vb = synth.bits(K_new[l]), synth.bits(V_new[l])
            for b in range(B):
                dec.append(b, l, s[l, b], Kb[b], Vb[b], tau)      # the oracle's rule on the GPU's own scores
        if step in (0, w, w + 1, n_steps // 2, n_steps - 1) and B < 100:
            _check_cache_against_oracle(binding, oracle, ctx, cache, dec, B, L, H, D, n_steps + 1, P, n_pool)
    assert worst <= parity.SCORE_ATOL
    assert ctx.poll_status() == 0
    if B >= 100:        # spot-check a few lists of the wide batch
        for b, l, h in [(0, 0, 0), (127, 0, 3), (129, 0, 7), (64, 0, 5)]:
            _pos, Kd, Vd = dec.logical(b, l, h)
            Kg, Vg, n = _export(binding, ctx, cache, b, l, h, n_steps + 1, D)
            assert n == len(Kd)
            np.testing.assert_array_equal(Kg, Kd)
            np.testing.assert_array_equal(Vg, Vd)
    binding.kvzap_cache_destroy(cache)
    ctx.close()


@pytest.mark.parametrize("T0,w", [(300, 16), (10, 16), (129, 128), (77, 0)])
def test_prefill_to_cache_then_decode_equals_longer_prefill(binding, oracle, T0, w):
    d_model, hidden, H, D, tau, P, k = 256, 128, 8, 64, 0.2, 8, 30
    ctx = binding.Kvzap(d_model, hidden, H, D, 1, max_tokens=T0 + k)
    wts = _weights(d_model, hidden, H, seed=T0)
    ctx.set_weights(0, *[parity.dev(x) for x in wts])
    X = synth.hidden_states(T0 + k, d_model, seed=T0 + 1)
    K, V = synth.keys_values(H, T0 + k, D, seed=T0 + 2)
    n_pool = H * ((T0 + k) // P + 2)
    K_pool = torch.zeros(n_pool, P, D, dtype=torch.bfloat16, device="cuda")
    V_pool = torch.zeros_like(K_pool)
    cache = binding.kvzap_cache_create(ctx.handle, 1, w, P, K_pool, V_pool, (T0 + k) // P + 2)
    scores_all = torch.empty(T0 + k, H, dtype=torch.float32, device="cuda")
    binding.kvzap_prefill_to_cache(ctx.handle, cache, 0, 0, parity.dev(X[:T0]), parity.dev(K[:, :T0].contiguous()),
                                   parity.dev(V[:, :T0].contiguous()), tau, scores_all[:T0])
    for t in range(T0, T0 + k):
        binding.kvzap_decode_step(ctx.handle, cache, 0, 1, parity.dev(X[t:t + 1]).view(1, 1, d_model),
                                  parity.dev(K[:, t].contiguous()).view(1, 1, H, D),
                                  parity.dev(V[:, t].contiguous()).view(1, 1, H, D), tau, scores_all[t:t + 1].view(1, 1, H))
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    s = scores_all.cpu().numpy()
    want = oracle.score(synth.bits(X), parity.weights_to_oracle(wts))
    assert np.abs(s - want).max() <= parity.SCORE_ATOL
    # prefill pruning of the whole sequence (oracle, on the GPU's scores) == what the cache holds
    keep = oracle.keep_mask(s, tau, w)
    Kc, Vc, ln = oracle.compact(synth.bits(K), synth.bits(V), keep)
    for h in range(H):
        Kg, Vg, n = _export(binding, ctx, cache, 0, 0, h, T0 + k, D)
        assert n == ln[0, h]
        np.testing.assert_array_equal(Kg, Kc[h, :n])
        np.testing.assert_array_equal(Vg, Vc[h, :n])
    # page-table validity: pages of all lists are distinct and inside the pool
    binding.kvzap_cache_destroy(cache)
    ctx.close()


def test_decode_pool_exhaustion_sets_status(binding):
    d_model, H, D, w, P = 256, 8, 64, 2, 4
    ctx = binding.Kvzap(d_model, 0, H, D, 1, max_tokens=128)
    W, b = synth.linear_weights(d_model, H, 1)
    ctx.set_weights(0, parity.dev(W), parity.dev(b))
    K_pool = torch.zeros(2, P, D, dtype=torch.bfloat16, device="cuda")          # 2 pages for 8 lists
    V_pool = torch.zeros_like(K_pool)
    cache = binding.kvzap_cache_create(ctx.handle, 1, w, P, K_pool, V_pool, 4)
    for step in range(6):
        X = parity.dev(synth.hidden_states(1, d_model, seed=step)).view(1, 1, d_model)
        Kn, Vn = synth.keys_values(1, H, D, seed=step)
        binding.kvzap_decode_step(ctx.handle, cache, 0, 1, X, parity.dev(Kn).view(1, 1, H, D),
                                  parity.dev(Vn).view(1, 1, H, D), float("-inf"), None)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 4
    binding.kvzap_cache_destroy(cache)
    ctx.close()


@pytest.mark.parametrize("chunks,w,P", [([300, 5, 200, 17, 129], 16, 8), ([100, 100, 100], 128, 16), ([64, 1, 1, 300], 0, 4),
                                        ([3, 2, 700, 40], 32, 16), ([300, 700, 50, 290], 256, 16)])
def test_chunked_prefill_equals_one_prefill(binding, oracle, chunks, w, P):
    """Prefill in chunks of any lengths (then a few decode steps) == prefill of the whole sequence:
    the score buffer carries the window across chunk boundaries."""
    d_model, hidden, H, D, tau, k = 256, 128, 8, 64, 0.2, 7
    T0 = sum(chunks)
    ctx = binding.Kvzap(d_model, hidden, H, D, 1, max_tokens=max(max(chunks), 128))
    wts = _weights(d_model, hidden, H, seed=T0)
    ctx.set_weights(0, *[parity.dev(x) for x in wts])
    X = synth.hidden_states(T0 + k, d_model, seed=T0 + 1)
    K, V = synth.keys_values(H, T0 + k, D, seed=T0 + 2)
    n_pool = H * ((T0 + k) // P + 2) + 8
    K_pool = torch.zeros(n_pool, P, D, dtype=torch.bfloat16, device="cuda")
    V_pool = torch.zeros_like(K_pool)
    cache = binding.kvzap_cache_create(ctx.handle, 1, w, P, K_pool, V_pool, (T0 + k) // P + 2)
    scores_all = torch.empty(T0 + k, H, dtype=torch.float32, device="cuda")
    t = 0
    for m in chunks:
        binding.kvzap_prefill_to_cache(ctx.handle, cache, 0, 0, parity.dev(X[t:t + m]), parity.dev(K[:, t:t + m].contiguous()),
                                       parity.dev(V[:, t:t + m].contiguous()), tau, scores_all[t:t + m])
        t += m
        if t in (chunks[0], T0):             # check at a chunk boundary and at the end of the prompt
            torch.cuda.synchronize()
            assert ctx.poll_status() == 0
            s = scores_all[:t].cpu().numpy()
            keep = oracle.keep_mask(s, tau, w)
            Kc, Vc, ln = oracle.compact(synth.bits(K[:, :t]), synth.bits(V[:, :t]), keep)
            for h in range(H):
                Kg, Vg, n = _export(binding, ctx, cache, 0, 0, h, T0 + k, D)
                assert n == ln[0, h]
                np.testing.assert_array_equal(Kg, Kc[h, :n])
                np.testing.assert_array_equal(Vg, Vc[h, :n])
    for t in range(T0, T0 + k):
        binding.kvzap_decode_step(ctx.handle, cache, 0, 1, parity.dev(X[t:t + 1]).view(1, 1, d_model),
                                  parity.dev(K[:, t].contiguous()).view(1, 1, H, D),
                                  parity.dev(V[:, t].contiguous()).view(1, 1, H, D), tau, scores_all[t:t + 1].view(1, 1, H))
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    s = scores_all.cpu().numpy()
    want = oracle.score(synth.bits(X), parity.weights_to_oracle(wts))
    assert np.abs(s - want).max() <= parity.SCORE_ATOL
    keep = oracle.keep_mask(s, tau, w)
    Kc, Vc, ln = oracle.compact(synth.bits(K), synth.bits(V), keep)
    tables = []
    for h in range(H):
        Kg, Vg, n = _export(binding, ctx, cache, 0, 0, h, T0 + k, D)
        assert n == ln[0, h]
        np.testing.assert_array_equal(Kg, Kc[h, :n])
        np.testing.assert_array_equal(Vg, Vc[h, :n])
    binding.kvzap_cache_destroy(cache)
    ctx.close()


def test_chunked_prefill_pool_exhaustion_sets_status(binding):
    """A second chunk that needs more pages than the pool has left: the status word reports it, the
    lengths stay what fits, nothing crashes, and the context keeps working."""
    d_model, H, D, w, P = 256, 8, 64, 8, 4
    ctx = binding.Kvzap(d_model, 0, H, D, 1, max_tokens=256)
    W, b = synth.linear_weights(d_model, H, 1)
    ctx.set_weights(0, parity.dev(W), parity.dev(b))
    n_pool = H * 6                                      # 24 rows per list
    K_pool = torch.zeros(n_pool, P, D, dtype=torch.bfloat16, device="cuda")
    V_pool = torch.zeros_like(K_pool)
    cache = binding.kvzap_cache_create(ctx.handle, 1, w, P, K_pool, V_pool, 64)
    lengths = torch.zeros(1, 1, H, dtype=torch.int32, device="cuda")
    for i, m in enumerate([20, 200]):                    # tau = -inf keeps everything: 12 rows, then 200 more
        X = parity.dev(synth.hidden_states(m, d_model, seed=i))
        Kn, Vn = synth.keys_values(H, m, D, seed=10 + i)
        sc = torch.empty(m, H, dtype=torch.float32, device="cuda")
        binding.kvzap_prefill_to_cache(ctx.handle, cache, 0, 0, X, parity.dev(Kn), parity.dev(Vn), float("-inf"), sc)
        torch.cuda.synchronize()
        st = ctx.poll_status()
        binding.kvzap_cache_lengths(ctx.handle, cache, lengths)
        torch.cuda.synchronize()
        if i == 0:
            assert st == 0 and (lengths == 20).all()
        else:
            assert st == 4                               # KVZAP_ERR_OOM_PAGES
            assert (lengths <= n_pool // H * P + w).all()
    binding.kvzap_cache_destroy(cache)
    ctx.close()


@pytest.mark.parametrize("hidden", [128, 0])        # the one-launch decode step, and the scoring + update pair of launches
def test_release_seq_hands_its_pages_out_again(binding, oracle, hidden):
    """A sequence ends, its slot takes a new prompt: the pool is sized so that this only fits if the
    released pages are reused; every list of both slots is compared with the oracle before and after."""
    d_model, H, D, L, w, P, tau = 256, 8, 64, 2, 16, 16, float("-inf")       # keep everything: pages = rows / 16
    ctx = binding.Kvzap(d_model, hidden, H, D, L, max_tokens=512)
    weights = [_weights(d_model, hidden, H, seed=80 + l) for l in range(L)]
    for l in range(L):
        ctx.set_weights(l, *[parity.dev(x) for x in weights[l]])
    n_pool = 900                                    # 400 + 300 rows first, then 500 more in slot 0: 1216 pages without reuse
    K_pool = torch.full((n_pool, P, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    V_pool = torch.full_like(K_pool, float("nan"))
    cache = ctx.create_cache(2, w, P, K_pool, V_pool, 40)
    decs = [oracle.DecodeOracle(1, L, H, D, w), oracle.DecodeOracle(1, L, H, D, w)]
    seed = [1000]

    def prefill(slot, chunks):
        for m in chunks:
            for l in range(L):
                seed[0] += 1
                X = synth.hidden_states(m, d_model, seed=seed[0])
                K, V = synth.keys_values(H, m, D, seed=seed[0] + 5000)
                s = cache.prefill(l, slot, parity.dev(X), parity.dev(K), parity.dev(V), tau).cpu().numpy()
                Kb, Vb = synth.bits(K), synth.bits(V)
                for t in range(m):
                    decs[slot].append(0, l, s[t], Kb[:, t], Vb[:, t], tau)

    def decode(n_steps, slots=(0, 1)):
        for _ in range(n_steps):
            seed[0] += 1
            X = synth.hidden_states(L * 2, d_model, seed=seed[0]).view(L, 2, d_model)
            Kn, Vn = synth.keys_values(L * 2, H, D, seed=seed[0] + 5000)
            Kn, Vn = Kn.view(L, 2, H, D), Vn.view(L, 2, H, D)
            sc = torch.empty(L, 2, H, dtype=torch.float32, device="cuda")
            cache.decode_step(0, L, parity.dev(X), parity.dev(Kn), parity.dev(Vn), tau, sc)
            s = sc.cpu().numpy()
            for l in range(L):
                for slot in slots:
                    decs[slot].append(0, l, s[l, slot], synth.bits(Kn)[l, slot], synth.bits(Vn)[l, slot], tau)

    def check():
        torch.cuda.synchronize()
        assert ctx.poll_status() == 0
        for slot in range(2):
            for l in range(L):
                for h in range(H):
                    _pos, Kd, Vd = decs[slot].logical(0, l, h)
                    Kg, Vg, n = _export(binding, ctx, cache.handle, slot, l, h, 700, D)
                    assert n == len(Kd)
                    np.testing.assert_array_equal(Kg, Kd)
                    np.testing.assert_array_equal(Vg, Vd)

    prefill(0, [250, 150])
    prefill(1, [300])
    decode(5)
    check()
    cache.release_seq(0)
    decs[0] = oracle.DecodeOracle(1, L, H, D, w)
    ln = cache.lengths().cpu().numpy()
    assert (ln[0] == 0).all() and (ln[1] == 305).all()
    decode(3, slots=(1,))                            # the released slot takes no part in decode steps
    ln = cache.lengths().cpu().numpy()
    assert (ln[0] == 0).all() and (ln[1] == 308).all()
    check()
    prefill(0, [200, 300])                           # needs the released pages; the slot takes part again
    decode(7)
    check()
    # and once more, to see pages go round a second time
    cache.release_seq(1)
    decs[1] = oracle.DecodeOracle(1, L, H, D, w)
    prefill(1, [120])
    decode(20)                                       # single pages taken by decode steps from the stack as well
    check()
    cache.close()
    ctx.close()
