"""Decode steps on caches that already hold long prefixes, and decode steps queued directly behind
prompt chunks, against the decode oracle.

The benchmark's decode workload installs prefixes of 4096..32768 rows per list (kvzap_cache_import)
and then decodes, so every kept row that leaves the window is appended at row `prefix_len` of a list
whose page table is already thousands of entries long.  Here the same state is built at a size that
memory can back in full (4 sequences, 2 layers), decoded for w + 72 steps enqueued back to back, and
every list is compared bit for bit with the oracle's rule (caption of Algorithm 1: a token is decided by
its buffered score when it leaves the window; Method, "KVzap": dropped iff score < tau) applied to the
GPU's own scores; the page tables are checked for validity (any unique in-range page is a correct
allocation).
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


def _export(binding, ctx, cache, b, l, h, cap, D):
    K_out = torch.zeros(cap, D, dtype=torch.bfloat16, device="cuda")
    V_out = torch.zeros(cap, D, dtype=torch.bfloat16, device="cuda")
    n = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.kvzap_cache_export(ctx.handle, cache, b, l, h, K_out, V_out, n)
    torch.cuda.synchronize()
    n = int(n.item())
    return synth.bits(K_out[:n]), synth.bits(V_out[:n]), n


def _snapshot(binding, ctx, cache, n_lists, max_pages):
    prefix = torch.zeros(n_lists, dtype=torch.int32, device="cuda")
    table = torch.zeros(n_lists, max_pages, dtype=torch.int32, device="cuda")
    cursor = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.kvzap_cache_snapshot(ctx.handle, cache, prefix, table, cursor)
    torch.cuda.synchronize()
    return prefix.cpu().numpy(), table.cpu().numpy(), int(cursor.item())


def _owned_pages(prefix, table, P):
    """All (list, page) pairs in use; asserts that no page is owned twice."""
    owned = []
    for li in range(len(prefix)):
        n_pages = -(-int(prefix[li]) // P)
        owned.append(table[li, :n_pages])
    flat = np.concatenate(owned) if owned else np.zeros(0, dtype=np.int32)
    assert len(np.unique(flat)) == len(flat), "a pool page is owned by two lists (or twice by one)"
    return flat


@pytest.mark.parametrize("hidden,trusted", [(512, True), (512, False), (0, True)])
def test_imported_long_prefixes_then_decode_with_evictions(binding, oracle, hidden, trusted):
    d_model, H, D, w, P, B, L, tau = 4096, 8, 128, 128, 16, 4, 2, 0.43
    n_steps = w + 72
    ctx = binding.Kvzap(d_model, hidden, H, D, L, max_tokens=128, trusted_producers=trusted)
    weights = []
    for l in range(L):
        wts = (synth.mlp_weights(d_model, hidden, H, 7300 + l, "cuda") if hidden
               else synth.linear_weights(d_model, H, 7300 + l, "cuda"))
        weights.append(wts)
        ctx.set_weights(l, *wts)
    n_lists = B * L * H
    rng = np.random.default_rng(505)
    prefix = rng.integers(4096, 32768 + 1, size=n_lists).astype(np.int32)
    prefix[0], prefix[1], prefix[2] = 4096, 32768, 4096 + 15          # a full last page, the maximum, a page one short of full
    pages_of = (prefix + P - 1) // P
    first = np.concatenate([[0], np.cumsum(pages_of)[:-1]]).astype(np.int64)
    next_free = int(pages_of.sum())
    grow = n_steps // P + 2
    n_pool = next_free + n_lists * grow
    max_pages = int(pages_of.max()) + grow
    g = torch.Generator(device="cuda").manual_seed(99)
    K_pool = torch.randn(n_pool, P, D, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    V_pool = torch.randn(n_pool, P, D, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    table_np = np.full((n_lists, max_pages), -1, dtype=np.int32)
    for li in range(n_lists):
        table_np[li, :pages_of[li]] = first[li] + np.arange(pages_of[li])
    # what the lists hold before decoding: their imported rows, in order
    Kp_bits, Vp_bits = synth.bits(K_pool).reshape(-1, D), synth.bits(V_pool).reshape(-1, D)
    imported = []
    for li in range(n_lists):
        r0 = int(first[li]) * P
        imported.append((Kp_bits[r0:r0 + prefix[li]].copy(), Vp_bits[r0:r0 + prefix[li]].copy()))
    del Kp_bits, Vp_bits
    cache = binding.kvzap_cache_create(ctx.handle, B, w, P, K_pool, V_pool, max_pages)
    binding.kvzap_cache_import(ctx.handle, cache, torch.from_numpy(prefix).cuda(), torch.from_numpy(table_np).cuda(), next_free)

    Xs, Ks, Vs = [], [], []
    for step in range(n_steps):
        Xs.append(synth.hidden_states(L * B, d_model, 9100 + step, "cuda").view(L, B, d_model))
        Kn, Vn = synth.keys_values(L * B, H, D, 9600 + step, "cuda")
        Ks.append(Kn.view(L, B, H, D))
        Vs.append(Vn.view(L, B, H, D))
    scores_all = torch.empty(n_steps, L, B, H, dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    for step in range(n_steps):                       # back to back, a scores buffer of its own per step
        binding.kvzap_decode_step(ctx.handle, cache, 0, L, Xs[step], Ks[step], Vs[step], tau, scores_all[step])
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    s_all = scores_all.cpu().numpy()
    for step, l in [(0, 0), (w, 1), (n_steps - 1, 0)]:
        want = oracle.score(synth.bits(Xs[step][l]), parity.weights_to_oracle(tuple(t.cpu() for t in weights[l])))
        assert np.abs(s_all[step, l] - want).max() <= parity.SCORE_ATOL

    dec = oracle.DecodeOracle(B, L, H, D, w)
    for step in range(n_steps):
        Kb, Vb = synth.bits(Ks[step]), synth.bits(Vs[step])          # [L, B, H, D]
        for l in range(L):
            for b in range(B):
                dec.append(b, l, s_all[step, l, b], Kb[l, b], Vb[l, b], tau)
    lengths = torch.zeros(B, L, H, dtype=torch.int32, device="cuda")
    binding.kvzap_cache_lengths(ctx.handle, cache, lengths)
    ln = lengths.cpu().numpy()
    n_joined = 0
    for b in range(B):
        for l in range(L):
            for h in range(H):
                li = (b * L + l) * H + h
                _pos, Kd, Vd = dec.logical(b, l, h)
                want_K = np.concatenate([imported[li][0], Kd])
                want_V = np.concatenate([imported[li][1], Vd])
                assert ln[b, l, h] == len(want_K)
                Kg, Vg, n = _export(binding, ctx, cache, b, l, h, len(want_K) + 8, D)
                assert n == len(want_K)
                np.testing.assert_array_equal(Kg, want_K)
                np.testing.assert_array_equal(Vg, want_V)
                n_joined += len(dec.prefix[b][l][h])
    assert n_joined > n_lists * 5                      # rows really joined the prefixes (about a quarter of 72 per list)
    # page tables: the imported entries are untouched, every new page lies between the imported cursor
    # and the present one, no page is owned twice
    pre, tab, cursor = _snapshot(binding, ctx, cache, n_lists, max_pages)
    flat = _owned_pages(pre, tab, P)
    assert flat.min() >= 0 and flat.max() < cursor <= n_pool
    for li in range(n_lists):
        b, l, h = li // (L * H), (li // H) % L, li % H
        assert pre[li] == prefix[li] + len(dec.prefix[b][l][h])
        np.testing.assert_array_equal(tab[li, :pages_of[li]], table_np[li, :pages_of[li]])
        new = tab[li, pages_of[li]:-(-int(pre[li]) // P)]
        assert (new >= next_free).all()
    binding.kvzap_cache_destroy(cache)
    ctx.close()


def test_prompt_into_released_slot_then_decode_steps_back_to_back(binding, oracle):
    """A launch of 20 layers (80 CTAs: more than half of the SMs, the size from which consecutive fused
    decode steps overlap) on a context that trusts its producers.  A sequence is released, the slot is
    given a new prompt layer by layer, and decode steps follow with no host synchronisation anywhere:
    the first of them is queued directly behind the prompt chunk's page assignment and compaction and
    must not touch the page allocator or the lists before those have finished."""
    d_model, hidden, H, D, w, P, B, L, tau = 1024, 512, 8, 64, 32, 8, 6, 20, 0.2
    ctx = binding.Kvzap(d_model, hidden, H, D, L, max_tokens=512, trusted_producers=True)
    weights = []
    for l in range(L):
        wts = synth.mlp_weights(d_model, hidden, H, 8100 + l, "cuda", 0.3)
        weights.append(wts)
        ctx.set_weights(l, *wts)
    n_lists = B * L * H
    rng = np.random.default_rng(11)
    T0 = [int(rng.integers(120, 400)) for _ in range(B)]
    T_new = 333
    n_pool = (sum(T0) + T_new) * L * H // P + 4 * n_lists
    max_pages = (max(T0 + [T_new]) + 200) // P + 2
    K_pool = torch.zeros(n_pool, P, D, dtype=torch.bfloat16, device="cuda")
    V_pool = torch.zeros_like(K_pool)
    cache = binding.kvzap_cache_create(ctx.handle, B, w, P, K_pool, V_pool, max_pages)
    dec = oracle.DecodeOracle(B, L, H, D, w)
    pending = []                                       # (kind, data) replayed on the oracle after the GPU has run

    def prompt(b, T, seed):
        for l in range(L):
            X = synth.hidden_states(T, d_model, seed + l, "cuda")
            K, V = synth.keys_values(H, T, D, seed + 100 + l, "cuda")
            sc = torch.empty(T, H, dtype=torch.float32, device="cuda")
            binding.kvzap_prefill_to_cache(ctx.handle, cache, l, b, X, K, V, tau, sc)
            pending.append(("prompt", (b, l, sc, K, V)))

    def steps(n, seed):
        for i in range(n):
            X = synth.hidden_states(L * B, d_model, seed + i, "cuda").view(L, B, d_model)
            Kn, Vn = synth.keys_values(L * B, H, D, seed + 500 + i, "cuda")
            sc = torch.empty(L, B, H, dtype=torch.float32, device="cuda")
            binding.kvzap_decode_step(ctx.handle, cache, 0, L, X, Kn.view(L, B, H, D), Vn.view(L, B, H, D), tau, sc)
            pending.append(("step", (sc, Kn.view(L, B, H, D), Vn.view(L, B, H, D))))

    for b in range(B):
        prompt(b, T0[b], 1000 * (b + 1))
    steps(12, 50000)
    binding.kvzap_cache_release_seq(ctx.handle, cache, 2)
    pending.append(("release", 2))
    prompt(2, T_new, 77000)
    steps(w + 20, 60000)                               # directly behind the last layer's prompt chunk
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0

    for kind, data in pending:
        if kind == "prompt":
            b, l, sc, K, V = data
            dec.seed_prefill(b, l, sc.cpu().numpy(), synth.bits(K), synth.bits(V), tau)
        elif kind == "release":
            for l in range(L):
                for h in range(H):
                    dec.prefix[data][l][h].clear()
                    dec.window[data][l][h].clear()
                dec.n_tokens[data, l] = 0
        else:
            sc, Kn, Vn = data
            s, Kb, Vb = sc.cpu().numpy(), synth.bits(Kn), synth.bits(Vn)
            for l in range(L):
                for b in range(B):
                    dec.append(b, l, s[l, b], Kb[l, b], Vb[l, b], tau)
    lengths = torch.zeros(B, L, H, dtype=torch.int32, device="cuda")
    binding.kvzap_cache_lengths(ctx.handle, cache, lengths)
    ln = lengths.cpu().numpy()
    cap = max(T0 + [T_new]) + 200
    for b in range(B):
        for l in range(L):
            for h in range(H):
                assert ln[b, l, h] == dec.length(b, l, h), (b, l, h)
    rng = np.random.default_rng(3)
    sample = {(2, l, h) for l in range(L) for h in (0, 7)} | {(int(rng.integers(B)), int(rng.integers(L)), int(rng.integers(H))) for _ in range(60)}
    for (b, l, h) in sorted(sample):
        _pos, Kd, Vd = dec.logical(b, l, h)
        Kg, Vg, n = _export(binding, ctx, cache, b, l, h, cap, D)
        assert n == len(Kd)
        np.testing.assert_array_equal(Kg, Kd)
        np.testing.assert_array_equal(Vg, Vd)
    pre, tab, cursor = _snapshot(binding, ctx, cache, n_lists, max_pages)
    flat = _owned_pages(pre, tab, P)
    assert flat.min() >= 0 and flat.max() < cursor <= n_pool
    binding.kvzap_cache_destroy(cache)
    ctx.close()


def test_bounded_wait_of_the_fused_step_runs_out_and_the_cache_survives(binding, oracle):
    """Failure detection without a fault: the host's step count is skewed by one, so every cluster of the
    next fused decode step waits for a step that never ran.  With a short limit the wait gives up: the
    kernel returns, the status word reads KVZAP_ERR_TIMEOUT, nothing of the cache has changed, and after
    the poll (which clears the step counters) decoding goes on as if the failed step had not been made."""
    d_model, hidden, H, D, w, P, B, L, tau = 256, 128, 8, 64, 8, 4, 3, 2, 0.1
    ctx = binding.Kvzap(d_model, hidden, H, D, L, max_tokens=128)
    all_w = []
    for l in range(L):
        wts = synth.mlp_weights(d_model, hidden, H, 60 + l, "cuda", 0.3)
        all_w.append(wts)
        ctx.set_weights(l, *wts)
    n_steps = 30
    n_pool = B * L * H * (n_steps // P + 2)
    K_pool = torch.zeros(n_pool, P, D, dtype=torch.bfloat16, device="cuda")
    V_pool = torch.zeros_like(K_pool)
    max_pages = n_steps // P + 2
    cache = binding.kvzap_cache_create(ctx.handle, B, w, P, K_pool, V_pool, max_pages)
    dec = oracle.DecodeOracle(B, L, H, D, w)

    def step(i, feed_oracle=True):
        X = synth.hidden_states(L * B, d_model, 3000 + i, "cuda").view(L, B, d_model)
        Kn, Vn = synth.keys_values(L * B, H, D, 4000 + i, "cuda")
        Kn, Vn = Kn.view(L, B, H, D), Vn.view(L, B, H, D)
        sc = torch.empty(L, B, H, dtype=torch.float32, device="cuda")
        launches = ctx.launch_count()
        binding.kvzap_decode_step(ctx.handle, cache, 0, L, X, Kn, Vn, tau, sc)
        assert ctx.launch_count() == launches + 1          # the one-launch (fused) step
        torch.cuda.synchronize()
        if feed_oracle:
            s, Kb, Vb = sc.cpu().numpy(), synth.bits(Kn), synth.bits(Vn)
            for l in range(L):
                for b in range(B):
                    dec.append(b, l, s[l, b], Kb[l, b], Vb[l, b], tau)

    def state():
        lengths = torch.zeros(B, L, H, dtype=torch.int32, device="cuda")
        binding.kvzap_cache_lengths(ctx.handle, cache, lengths)
        lists = [_export(binding, ctx, cache, b, l, h, n_steps + 1, D) for b in range(B) for l in range(L) for h in range(H)]
        pre, tab, cursor = _snapshot(binding, ctx, cache, B * L * H, max_pages)
        return lengths.cpu().numpy(), lists, pre, cursor

    for i in range(14):
        step(i)
    assert ctx.poll_status() == 0
    before = state()
    binding.kvzap_set_wait_limit(ctx.handle, 200000)          # a tenth of a millisecond
    binding.kvzap_cache_debug_skew_steps(cache, 1)
    step(14, feed_oracle=False)                               # every cluster gives up; the kernel returns
    assert ctx.poll_status() == 5                             # KVZAP_ERR_TIMEOUT, cleared by the poll
    assert ctx.poll_status() == 0
    after = state()
    np.testing.assert_array_equal(before[0], after[0])
    np.testing.assert_array_equal(before[2], after[2])
    assert before[3] == after[3]
    for (Ka, Va, na), (Kb_, Vb_, nb) in zip(before[1], after[1]):
        assert na == nb
        np.testing.assert_array_equal(Ka, Kb_)
        np.testing.assert_array_equal(Va, Vb_)
    for i in range(15, n_steps):                              # ordinary steps again
        step(i)
    assert ctx.poll_status() == 0
    for b in range(B):
        for l in range(L):
            for h in range(H):
                _pos, Kd, Vd = dec.logical(b, l, h)
                Kg, Vg, n = _export(binding, ctx, cache, b, l, h, n_steps + 1, D)
                assert n == len(Kd)
                np.testing.assert_array_equal(Kg, Kd)
                np.testing.assert_array_equal(Vg, Vd)
    with pytest.raises(binding.KvzapError):
        binding.kvzap_set_wait_limit(ctx.handle, 10)
    binding.kvzap_cache_destroy(cache)
    ctx.close()
