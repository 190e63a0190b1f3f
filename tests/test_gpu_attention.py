"""GPU parity for attention over the pruned cache, against the CPU oracle.

The cache content is driven exactly as in the decode tests (the decode oracle follows the
GPU's own scores, so both sides hold the same lists); the attention output of every list
is then compared with the oracle's softmax attention over the oracle's copy of that list.

Tolerance: products are exact in fp32, the softmax runs in fp32, probabilities are rounded
to bf16 (relative 2^-9) before the second product and the output is rounded to bf16 once
(relative 2^-9 of values of order one); ATTN_ATOL = 2e-2 covers both with room.
"""
import numpy as np
import pytest
import torch

from paper_2601_07891_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu

ATTN_ATOL = 2e-2


@pytest.fixture(scope="module")
def binding():
    from paper_2601_07891_b200 import binding as b
    b.load()
    return b


def _weights(d_model, hidden, H, seed):
    if hidden == 0:
        return synth.linear_weights(d_model, H, seed, "cpu", 0.3)
    return synth.mlp_weights(d_model, hidden, H, seed, "cpu", 0.3)


def _poisoned_pool(n_pool, P, D):
    """Pools start as NaN bit patterns: a row read past the end of a list would poison the output."""
    return torch.full((n_pool, P, D), float("nan"), dtype=torch.bfloat16, device="cuda")


def _check_attention(binding, oracle, ctx, cache, dec, L, B, H, G, D, seed):
    Q = synth.hidden_states(L * B * H * G, D, seed=seed).view(L, B, H * G, D)
    O = torch.full((L, B, H * G, D), 7.0, dtype=torch.bfloat16, device="cuda")
    scale = 1.0 / np.sqrt(D)
    binding.kvzap_decode_attention(ctx.handle, cache, 0, L, parity.dev(Q), scale, O)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    got = O.float().cpu().numpy()
    assert np.isfinite(got).all()
    Qb = synth.bits(Q)
    worst = 0.0
    for l in range(L):
        for b in range(B):
            for h in range(H):
                _pos, Kd, Vd = dec.logical(b, l, h)
                want = oracle.attention(Qb[l, b, h * G:(h + 1) * G], Kd, Vd, scale)
                worst = max(worst, float(np.abs(got[l, b, h * G:(h + 1) * G] - want).max()))
    assert worst <= ATTN_ATOL, worst
    return worst


@pytest.mark.parametrize("hidden,w,P,B,L,D,G", [
    (128, 16, 16, 3, 2, 64, 4),
    (0, 32, 16, 2, 1, 128, 4),
    (64, 0, 16, 2, 1, 128, 8),        # no window: a new token is decided at once
    (128, 16, 32, 5, 1, 128, 1),      # two tiles per page, one query head per KV head
])
def test_attention_after_decode_steps(binding, oracle, hidden, w, P, B, L, D, G):
    d_model, H, tau, n_steps = 256, 8, -0.2, 100
    ctx = binding.Kvzap(d_model, hidden, H, D, L, max_tokens=128, max_seqs=1)
    all_w = []
    for l in range(L):
        wts = _weights(d_model, hidden, H, seed=70 + l)
        all_w.append(wts)
        ctx.set_weights(l, *[parity.dev(x) for x in wts])
    max_pages = n_steps // P + 2
    n_pool = B * L * H * max_pages
    K_pool, V_pool = _poisoned_pool(n_pool, P, D), _poisoned_pool(n_pool, P, D)
    cache = binding.kvzap_cache_create(ctx.handle, B, w, P, K_pool, V_pool, max_pages)
    dec = oracle.DecodeOracle(B, L, H, D, w)
    for step in range(n_steps):
        X = synth.hidden_states(L * B, d_model, seed=3000 + step).view(L, B, d_model)
        K_new, V_new = synth.keys_values(L * B, H, D, seed=4000 + step)
        K_new, V_new = K_new.view(L, B, H, D), V_new.view(L, B, H, D)
        scores = torch.empty(L, B, H, dtype=torch.float32, device="cuda")
        binding.kvzap_decode_step(ctx.handle, cache, 0, L, parity.dev(X), parity.dev(K_new), parity.dev(V_new), tau, scores)
        torch.cuda.synchronize()
        s = scores.cpu().numpy()
        for l in range(L):
            Kb, Vb = synth.bits(K_new[l]), synth.bits(V_new[l])
            for b in range(B):
                dec.append(b, l, s[l, b], Kb[b], Vb[b], tau)
        # first token, a partly filled window, the step the window fills, ragged prefix tiles, the end
        if step in (0, 4, max(w - 1, 1), w + 1, 57, n_steps - 1):
            _check_attention(binding, oracle, ctx, cache, dec, L, B, H, G, D, seed=9000 + step)
    binding.kvzap_cache_destroy(cache)
    ctx.close()


@pytest.mark.parametrize("T0,w,D", [(1500, 128, 128), (700, 16, 64), (900, 256, 128)])
def test_attention_after_prefill_to_cache(binding, oracle, T0, w, D):
    """Long lists: many tiles per warp, so every pipeline stage is reused several times."""
    d_model, hidden, H, tau, P, G, k = 256, 128, 8, 0.0, 16, 4, 5
    ctx = binding.Kvzap(d_model, hidden, H, D, 1, max_tokens=T0 + k)
    wts = _weights(d_model, hidden, H, seed=T0)
    ctx.set_weights(0, *[parity.dev(x) for x in wts])
    X = synth.hidden_states(T0 + k, d_model, seed=T0 + 1)
    K, V = synth.keys_values(H, T0 + k, D, seed=T0 + 2)
    max_pages = (T0 + k) // P + 2
    n_pool = H * max_pages
    K_pool, V_pool = _poisoned_pool(n_pool, P, D), _poisoned_pool(n_pool, P, D)
    cache = binding.kvzap_cache_create(ctx.handle, 1, w, P, K_pool, V_pool, max_pages)
    scores_all = torch.empty(T0 + k, H, dtype=torch.float32, device="cuda")
    binding.kvzap_prefill_to_cache(ctx.handle, cache, 0, 0, parity.dev(X[:T0]), parity.dev(K[:, :T0].contiguous()),
                                   parity.dev(V[:, :T0].contiguous()), tau, scores_all[:T0])
    for t in range(T0, T0 + k):
        binding.kvzap_decode_step(ctx.handle, cache, 0, 1, parity.dev(X[t:t + 1]).view(1, 1, d_model),
                                  parity.dev(K[:, t].contiguous()).view(1, 1, H, D),
                                  parity.dev(V[:, t].contiguous()).view(1, 1, H, D), tau, scores_all[t:t + 1].view(1, 1, H))
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    # the lists are what prefill pruning of the whole sequence keeps (oracle, on the GPU's scores)
    s = scores_all.cpu().numpy()
    keep = oracle.keep_mask(s, tau, w)
    Kc, Vc, ln = oracle.compact(synth.bits(K), synth.bits(V), keep)
    Q = synth.hidden_states(H * G, D, seed=5).view(1, 1, H * G, D)
    O = torch.zeros(1, 1, H * G, D, dtype=torch.bfloat16, device="cuda")
    scale = 1.0 / np.sqrt(D)
    binding.kvzap_decode_attention(ctx.handle, cache, 0, 1, parity.dev(Q), scale, O)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    got = O.float().cpu().numpy()[0, 0]
    Qb = synth.bits(Q)[0, 0]
    for h in range(H):
        n = int(ln[0, h])
        assert n > 100
        want = oracle.attention(Qb[h * G:(h + 1) * G], Kc[h, :n], Vc[h, :n], scale)
        assert np.abs(got[h * G:(h + 1) * G] - want).max() <= ATTN_ATOL
    binding.kvzap_cache_destroy(cache)
    ctx.close()


def test_attention_empty_cache_and_argument_errors(binding):
    d_model, H, D, P, w = 256, 8, 128, 16, 16
    ctx = binding.Kvzap(d_model, 0, H, D, 1, max_tokens=128)
    W, b = synth.linear_weights(d_model, H, 1)
    ctx.set_weights(0, parity.dev(W), parity.dev(b))
    K_pool, V_pool = _poisoned_pool(32, P, D), _poisoned_pool(32, P, D)
    cache = binding.kvzap_cache_create(ctx.handle, 2, w, P, K_pool, V_pool, 2)
    Q = parity.dev(synth.hidden_states(2 * 32, D, seed=1).view(1, 2, 32, D))
    O = torch.full((1, 2, 32, D), 3.0, dtype=torch.bfloat16, device="cuda")
    binding.kvzap_decode_attention(ctx.handle, cache, 0, 1, Q, 0.1, O)       # nothing appended yet: zeros
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0 and (O == 0).all()
    with pytest.raises(binding.KvzapError):
        binding.kvzap_decode_attention(ctx.handle, cache, 0, 2, Q, 0.1, O)   # layer range
    with pytest.raises(binding.KvzapError):
        binding.kvzap_decode_attention(ctx.handle, cache, 0, 1, Q[:, :, :12].contiguous(), 0.1, O)   # 12 heads over 8
    with pytest.raises(binding.KvzapError):
        binding.kvzap_decode_attention(ctx.handle, cache, 0, 1, Q, -1.0, O)
    binding.kvzap_cache_destroy(cache)
    # a page size that is not a multiple of 16 is refused, not mis-read
    K7, V7 = _poisoned_pool(32, 7, D), _poisoned_pool(32, 7, D)
    cache7 = binding.kvzap_cache_create(ctx.handle, 2, w, 7, K7, V7, 4)
    with pytest.raises(binding.KvzapError):
        binding.kvzap_decode_attention(ctx.handle, cache7, 0, 1, Q, 0.1, O)
    binding.kvzap_cache_destroy(cache7)
    ctx.close()


@pytest.mark.parametrize("B,lo,hi", [(128, 1000, 8000), (300, 200, 2000)])
def test_attention_at_bench_size_sampled_lists(binding, oracle, B, lo, hi):
    """128 sequences x 8 KV heads with lists of 1k..8k pruned rows plus a full window of 128, the
    launch shape bench.py --attention times (one layer): sampled lists against the oracle.
    With 128 sequences every list is cut into parts, with 300 (2400 lists) each list is one CTA."""
    d_model, H, D, P, w, G = 256, 8, 128, 16, 128, 4
    ctx = binding.Kvzap(d_model, 0, H, D, 1, max_tokens=B)
    W, bias = synth.linear_weights(d_model, H, 3)
    ctx.set_weights(0, parity.dev(W), parity.dev(bias))
    n_lists = B * H
    rng = np.random.default_rng(99)
    prefix = rng.integers(lo, hi + 1, size=n_lists).astype(np.int32)
    prefix[:4] = [1, 15, 16, 17]                      # ragged first tiles
    pages_of = (prefix + P - 1) // P
    first = np.concatenate([[0], np.cumsum(pages_of)[:-1]]).astype(np.int64)
    n_pool, max_pages = int(pages_of.sum()), int(pages_of.max())
    Kp, Vp = synth.keys_values(1, n_pool * P, D, seed=123, device="cuda")          # [1, rows, D]
    K_pool, V_pool = Kp.view(n_pool, P, D), Vp.view(n_pool, P, D)
    # rows past a list's end inside its last page must not matter: overwrite them with NaN
    last_fill = prefix - (pages_of - 1) * P
    for li in range(0, n_lists, 37):
        pg = int(first[li] + pages_of[li] - 1)
        K_pool[pg, int(last_fill[li]):] = float("nan")
        V_pool[pg, int(last_fill[li]):] = float("nan")
    table = torch.from_numpy((first[:, None] + np.arange(max_pages)[None, :]).astype(np.int32)).cuda()
    cache = binding.kvzap_cache_create(ctx.handle, B, w, P, K_pool, V_pool, max_pages)
    binding.kvzap_cache_import(ctx.handle, cache, torch.from_numpy(prefix).cuda(), table, n_pool)
    n_steps = w + 3
    new_rows = []
    for step in range(n_steps):
        X = parity.dev(synth.hidden_states(B, d_model, seed=600 + step)).view(1, B, d_model)
        Kn, Vn = synth.keys_values(B, H, D, seed=700 + step)                       # [B, H, D]
        new_rows.append((synth.bits(Kn), synth.bits(Vn)))
        binding.kvzap_decode_step(ctx.handle, cache, 0, 1, X, parity.dev(Kn).view(1, B, H, D),
                                  parity.dev(Vn).view(1, B, H, D), float("inf"), None)    # nothing joins the prefix
    Q = synth.hidden_states(B * H * G, D, seed=8).view(1, B, H * G, D)
    O = torch.zeros(1, B, H * G, D, dtype=torch.bfloat16, device="cuda")
    scale = 1.0 / np.sqrt(D)
    binding.kvzap_decode_attention(ctx.handle, cache, 0, 1, parity.dev(Q), scale, O)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    got = O.float().cpu().numpy()[0]
    assert np.isfinite(got).all()
    Qb = synth.bits(Q)[0]
    Kp_bits, Vp_bits = synth.bits(K_pool.cpu()).reshape(-1, D), synth.bits(V_pool.cpu()).reshape(-1, D)
    sample = sorted(set([0, 1, 2, 3, 37, 74, n_lists - 1] + rng.integers(0, n_lists, 20).tolist()))
    for li in sample:
        b, h = li // H, li % H                         # one layer: list index = b * H + h
        r0 = int(first[li]) * P
        Kd = np.concatenate([Kp_bits[r0:r0 + int(prefix[li])]] + [new_rows[s][0][b, h][None] for s in range(n_steps - w, n_steps)])
        Vd = np.concatenate([Vp_bits[r0:r0 + int(prefix[li])]] + [new_rows[s][1][b, h][None] for s in range(n_steps - w, n_steps)])
        want = oracle.attention(Qb[b, h * G:(h + 1) * G], Kd, Vd, scale)
        assert np.abs(got[b, h * G:(h + 1) * G] - want).max() <= ATTN_ATOL, li
    binding.kvzap_cache_destroy(cache)
    ctx.close()


def test_decode_loop_step_then_attention_enqueued_back_to_back(binding, oracle):
    """The serving loop: decode step, attention, decode step, attention, ... all enqueued without a
    host synchronisation in between.  Every attention call must see exactly the cache its own step
    left (the next step, which may start early, must not disturb it)."""
    d_model, hidden, H, D, w, P, B, L, G, tau, n_steps = 256, 128, 8, 64, 16, 16, 6, 2, 4, 0.0, 70
    ctx = binding.Kvzap(d_model, hidden, H, D, L, max_tokens=128, max_seqs=1)
    all_w = []
    for l in range(L):
        wts = _weights(d_model, hidden, H, seed=90 + l)
        all_w.append(wts)
        ctx.set_weights(l, *[parity.dev(x) for x in wts])
    max_pages = n_steps // P + 2
    n_pool = B * L * H * max_pages
    K_pool, V_pool = _poisoned_pool(n_pool, P, D), _poisoned_pool(n_pool, P, D)
    cache = binding.kvzap_cache_create(ctx.handle, B, w, P, K_pool, V_pool, max_pages)
    scale = 1.0 / np.sqrt(D)
    Xs, Ks, Vs, Qs, Os, Ss = [], [], [], [], [], []
    for step in range(n_steps):
        Xs.append(parity.dev(synth.hidden_states(L * B, d_model, seed=100 + step).view(L, B, d_model)))
        Kn, Vn = synth.keys_values(L * B, H, D, seed=300 + step)
        Ks.append(parity.dev(Kn.view(L, B, H, D)))
        Vs.append(parity.dev(Vn.view(L, B, H, D)))
        Qs.append(parity.dev(synth.hidden_states(L * B * H * G, D, seed=500 + step).view(L, B, H * G, D)))
        Os.append(torch.zeros(L, B, H * G, D, dtype=torch.bfloat16, device="cuda"))
        Ss.append(torch.empty(L, B, H, dtype=torch.float32, device="cuda"))
    torch.cuda.synchronize()
    for step in range(n_steps):
        binding.kvzap_decode_step(ctx.handle, cache, 0, L, Xs[step], Ks[step], Vs[step], tau, Ss[step])
        binding.kvzap_decode_attention(ctx.handle, cache, 0, L, Qs[step], scale, Os[step])
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    dec = oracle.DecodeOracle(B, L, H, D, w)
    worst = 0.0
    for step in range(n_steps):
        s = Ss[step].cpu().numpy()
        Kb, Vb = synth.bits(Ks[step].cpu()), synth.bits(Vs[step].cpu())
        for l in range(L):
            for b in range(B):
                dec.append(b, l, s[l, b], Kb[l, b], Vb[l, b], tau)
        if step % 3 == 0 or step > n_steps - 4:
            got = Os[step].float().cpu().numpy()
            Qb = synth.bits(Qs[step].cpu())
            for l in range(L):
                for b in range(B):
                    for h in range(H):
                        _pos, Kd, Vd = dec.logical(b, l, h)
                        want = oracle.attention(Qb[l, b, h * G:(h + 1) * G], Kd, Vd, scale)
                        worst = max(worst, float(np.abs(got[l, b, h * G:(h + 1) * G] - want).max()))
    assert worst <= ATTN_ATOL, worst
    binding.kvzap_cache_destroy(cache)
    ctx.close()


def test_attention_without_window_and_with_one_row(binding, oracle):
    """w = 0 (nothing but the paged prefix) and lists of a single row."""
    d_model, H, D, P, G = 256, 8, 64, 16, 2
    ctx = binding.Kvzap(d_model, 0, H, D, 1, max_tokens=128)
    W, b = synth.linear_weights(d_model, H, 1)
    ctx.set_weights(0, parity.dev(W), parity.dev(b))
    K_pool, V_pool = _poisoned_pool(64, P, D), _poisoned_pool(64, P, D)
    cache = binding.kvzap_cache_create(ctx.handle, 2, 0, P, K_pool, V_pool, 4)
    dec = oracle.DecodeOracle(2, 1, H, D, 0)
    Q = synth.hidden_states(2 * H * G, D, seed=3).view(1, 2, H * G, D)
    O = torch.full((1, 2, H * G, D), 5.0, dtype=torch.bfloat16, device="cuda")
    for step in range(3):
        X = synth.hidden_states(2, d_model, seed=20 + step).view(1, 2, d_model)
        Kn, Vn = synth.keys_values(2, H, D, seed=30 + step)
        sc = torch.empty(1, 2, H, dtype=torch.float32, device="cuda")
        tau = float("-inf") if step == 0 else float("inf")         # the first token stays, later ones are dropped at once
        binding.kvzap_decode_step(ctx.handle, cache, 0, 1, parity.dev(X), parity.dev(Kn).view(1, 2, H, D),
                                  parity.dev(Vn).view(1, 2, H, D), tau, sc)
        torch.cuda.synchronize()
        s = sc.cpu().numpy()
        for bb in range(2):
            dec.append(bb, 0, s[0, bb], synth.bits(Kn)[bb], synth.bits(Vn)[bb], tau)
    binding.kvzap_decode_attention(ctx.handle, cache, 0, 1, parity.dev(Q), 0.125, O)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    got = O.float().cpu().numpy()[0]
    for bb in range(2):
        for h in range(H):
            _pos, Kd, Vd = dec.logical(bb, 0, h)
            assert len(Kd) == 1
            want = oracle.attention(synth.bits(Q)[0, bb, h * G:(h + 1) * G], Kd, Vd, 0.125)
            assert np.abs(got[bb, h * G:(h + 1) * G] - want).max() <= ATTN_ATOL
    binding.kvzap_cache_destroy(cache)
    ctx.close()
